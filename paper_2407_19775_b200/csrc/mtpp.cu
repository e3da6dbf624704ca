// mtpp.cu -- slicing topological orders into pipeline blocks (include/mtpp.h), one CTA per order.
//
// The segment cost of positions l..r of an order is never tabulated.  The dynamic programme
// walks r = 1..n, and for a fixed r the costs of ALL segments that end at r form one column,
// which follows from the column of r - 1 by adding the node v at position r:
//     work, sizeparam  += the node's;   peak = max(peak, sizeout(v));
//     in(l, r)  gains sizeout(u) for each producer u of v that lies before l and had no consumer
//               in l..r-1 yet, i.e. for l > max(pos(u), position of u's previous consumer);
//     out(l, r) gains sizeout(v) if v has consumers (they all come later), and loses sizeout(u)
//               for each producer u of v inside l..r whose last consumer is v.
// So a CTA keeps five running values per l (in the registers of the thread that owns l), the dp rows
// of every block count, and the positions of each node, its last consumer and its latest
// consumer so far: a few tens of kilobytes of shared memory, no global scratch.  Per step one barrier separates the column
// update from the minimisations, which warp kk does for block count kk.
#include "../../include/mtpp.h"
#include "bq_error.h"

#include <cuda_runtime.h>

#include <mutex>
#include <new>
#include <vector>

namespace {

constexpr int kSliceThreads = 256;
constexpr int kDecodeWarps = 4;
constexpr long long kInf = 0x7fffffffffffffffLL;
constexpr size_t kSliceSmemLimit = 226 * 1024;         // dynamic part of the 227 KB one CTA may take; the kernel's static words fit in the rest

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

struct DeviceGraph {
    int n;
    const int* pred_ptr;       // [n + 1]
    const int* pred;           // producers of each node
    const int* cons_ptr;       // [n + 1]
    const int* cons;           // consumers of each node
    const long long* work;
    const long long* sizeparam;
    const long long* sizeout;
};

__host__ __device__ inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Shared memory of slice_orders for (n, kmax): 64-bit arrays first, then 32-bit, then 16-bit.
struct SliceLayout {
    size_t f, dp, attr, pos, last, prev, pptr, pred, order, arg, total;
};
// `edges` > 0: the graph itself (attributes, producer lists) and the order are staged in shared memory too, so that the n
// dependent steps of the programme never wait for global memory; 0: they are read from global memory (graphs too large
// to fit beside the programme's own arrays).
__host__ __device__ inline SliceLayout slice_layout(int n, int kmax, int edges) {
    SliceLayout L;
    size_t o = 0;
    L.f = o;    o += size_t(n) * 8;                     // F(l, r) of the current r
    L.dp = o;   o += size_t(kmax) * (n + 1) * 8;        // dp[kk - 1][r]
    L.attr = o; o += edges > 0 ? size_t(3) * n * 8 : 0; // work | sizeparam | sizeout of the nodes
    L.pos = o;  o += size_t(n) * 4;                     // 1-based position of each node (0: not seen)
    L.last = o; o += size_t(n) * 4;                     // position of each node's last consumer (0: none)
    L.prev = o; o += size_t(n) * 4;                     // position of each node's latest consumer so far (0: none)
    L.pptr = o; o += edges > 0 ? size_t(n + 1) * 4 : 0; // producer lists: offsets ...
    L.pred = o; o += edges > 0 ? size_t(edges) * 4 : 0; // ... and entries
    L.order = o; o += edges > 0 ? size_t(n) * 4 : 0;    // the order itself
    L.arg = o;  o += size_t(kmax) * (n + 1) * 2;        // the cut that gave dp[kk - 1][r]
    L.total = (o + 15) / 16 * 16;
    return L;
}

template <int kOwned>                                               // first positions per thread: n <= kOwned * kSliceThreads
__global__ void __launch_bounds__(kSliceThreads)
slice_orders(DeviceGraph g, int staged_edges, const int* __restrict__ orders, int k, long long B, long long M, long long* __restrict__ cost_out,
             int* __restrict__ blocks_out, int* __restrict__ cuts_out, int* __restrict__ status_out) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int n = g.n;
    const int kmax = k < n ? k : n;
    const SliceLayout L = slice_layout(n, kmax, staged_edges);
    long long* F = reinterpret_cast<long long*>(smem + L.f);
    long long* dp = reinterpret_cast<long long*>(smem + L.dp);
    int* pos = reinterpret_cast<int*>(smem + L.pos);
    int* last = reinterpret_cast<int*>(smem + L.last);
    int* prev = reinterpret_cast<int*>(smem + L.prev);
    unsigned short* arg = reinterpret_cast<unsigned short*>(smem + L.arg);
    __shared__ int bad;

    const int p = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kSliceThreads / 32;
    const int* pi = orders + size_t(p) * n;
    const long long* a_work = g.work;
    const long long* a_param = g.sizeparam;
    const long long* a_out = g.sizeout;
    const int* pred_ptr = g.pred_ptr;
    const int* pred = g.pred;
    if (staged_edges > 0) {
        long long* sa = reinterpret_cast<long long*>(smem + L.attr);
        int* sp = reinterpret_cast<int*>(smem + L.pptr);
        int* sl = reinterpret_cast<int*>(smem + L.pred);
        int* so = reinterpret_cast<int*>(smem + L.order);
        for (int i = tid; i < n; i += kSliceThreads) { sa[i] = g.work[i]; sa[n + i] = g.sizeparam[i]; sa[2 * n + i] = g.sizeout[i]; so[i] = pi[i]; }
        for (int i = tid; i <= n; i += kSliceThreads) sp[i] = g.pred_ptr[i];
        for (int i = tid; i < staged_edges; i += kSliceThreads) sl[i] = g.pred[i];
        a_work = sa; a_param = sa + n; a_out = sa + 2 * n; pred_ptr = sp; pred = sl; pi = so;
    }

    // positions, and the check that the row is a topological order of this graph
    if (tid == 0) bad = 0;
    for (int i = tid; i < n; i += kSliceThreads) { pos[i] = 0; last[i] = 0; prev[i] = 0; }
    __syncthreads();
    for (int i = tid; i < n; i += kSliceThreads) {
        const int v = pi[i];
        if (v < 0 || v >= n) bad = 1;
        else if (atomicExch(&pos[v], i + 1) != 0) bad = 1;          // a node listed twice (so another one is missing)
    }
    __syncthreads();
    if (!bad) {
        for (int v = tid; v < n; v += kSliceThreads) {
            int lc = 0;
            for (int e = g.cons_ptr[v]; e < g.cons_ptr[v + 1]; ++e) {
                const int pc = pos[g.cons[e]];
                if (pc <= pos[v]) bad = 1;                           // a consumer before its producer
                lc = pc > lc ? pc : lc;
            }
            last[v] = lc;
        }
    }
    __syncthreads();
    if (bad) {
        if (tid == 0) { cost_out[p] = -1; blocks_out[p] = 0; status_out[p] = 1; }
        for (int j = tid; j < k; j += kSliceThreads) cuts_out[size_t(p) * k + j] = 0;
        return;
    }

    long long cw[kOwned], cp[kOwned], ck[kOwned], ci[kOwned], co[kOwned];
#pragma unroll
    for (int j = 0; j < kOwned; ++j) { cw[j] = 0; cp[j] = 0; ck[j] = 0; ci[j] = 0; co[j] = 0; }
    for (int r = 1; r <= n; ++r) {
        const int v = pi[r - 1];
        const int pb = pred_ptr[v], pe = pred_ptr[v + 1];
        const long long so_v = a_out[v], w_v = a_work[v], pa_v = a_param[v];
        const long long gain_out = (last[v] != 0) ? so_v : 0;            // v has consumers (they all come later)
        // the column of r: thread t owns the first positions l = t + 1, t + 257, ... and keeps their five running values in registers
#pragma unroll
        for (int j = 0; j < kOwned; ++j) {
            const int l = tid + 1 + j * kSliceThreads;
            if (l > r) continue;
            if (l == r) { cw[j] = 0; cp[j] = 0; ck[j] = 0; ci[j] = 0; co[j] = 0; }
            cw[j] += w_v;
            cp[j] += pa_v;
            ck[j] = so_v > ck[j] ? so_v : ck[j];
            co[j] += gain_out;
            for (int e = pb; e < pe; ++e) {
                const int u = pred[e];
                const int pu = pos[u], pc = prev[u];
                const long long so_u = a_out[u];
                if (l > (pu > pc ? pu : pc)) ci[j] += so_u;          // u lies before l and nothing in l..r-1 read it
                if (last[u] == r && pu >= l) co[j] -= so_u;           // u is inside and v was its last consumer
            }
            const long long excess = cp[j] + ck[j] - M;
            F[l - 1] = ci[j] + B * cw[j] + (excess > 0 ? excess : 0) + ck[j] + co[j];
        }
        __syncthreads();
        // dp[kk][r] = min over l of max(dp[kk - 1][l], F(l + 1, r)); the earlier l on equal values
        for (int kk = warp + 1; kk <= kmax; kk += kWarps) {
            long long best = kInf;
            int where = 0;
            if (kk == 1) {
                best = F[0];
            } else if (r >= kk) {
                const long long* below = dp + size_t(kk - 2) * (n + 1);
                for (int l = kk - 1 + lane; l < r; l += 32) {
                    const long long a = below[l], b = F[l];
                    const long long cand = a > b ? a : b;
                    if (cand < best) { best = cand; where = l; }     // l ascends within a lane: strict < keeps the earlier one
                }
                // the warp's smallest (value, position) pair by three 32-bit reductions: the high words, then the low words
                // among the lanes that hold the smallest high word, then the positions among the lanes that hold the smallest value
                const unsigned hi = unsigned(static_cast<unsigned long long>(best) >> 32), lo = unsigned(static_cast<unsigned long long>(best));
                const unsigned mh = __reduce_min_sync(0xffffffffu, hi);
                const unsigned ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
                const unsigned mi = __reduce_min_sync(0xffffffffu, (hi == mh && lo == ml) ? unsigned(where) : 0x7fffffffu);
                best = static_cast<long long>((static_cast<unsigned long long>(mh) << 32) | ml);
                where = int(mi);
            }
            if (lane == 0) {
                dp[size_t(kk - 1) * (n + 1) + r] = best;
                arg[size_t(kk - 1) * (n + 1) + r] = static_cast<unsigned short>(where);
            }
        }
        if (tid == kSliceThreads - 1) {                              // v has now been seen as a consumer of its producers
            for (int e = pb; e < pe; ++e) prev[pred[e]] = r;
        }
        __syncthreads();
    }

    if (tid == 0) {
        int best_k = 1;
        for (int kk = 2; kk <= kmax; ++kk)
            if (dp[size_t(kk - 1) * (n + 1) + n] < dp[size_t(best_k - 1) * (n + 1) + n]) best_k = kk;
        cost_out[p] = dp[size_t(best_k - 1) * (n + 1) + n];
        blocks_out[p] = best_k;
        status_out[p] = 0;
        int r = n;
        for (int kk = best_k; kk >= 1; --kk) {
            cuts_out[size_t(p) * k + kk - 1] = r;
            r = arg[size_t(kk - 1) * (n + 1) + r];
        }
        for (int j = best_k; j < k; ++j) cuts_out[size_t(p) * k + j] = 0;
    }
}

// One warp per key vector.  Per step the lanes look through the nodes for the ready one with the
// highest key (equal keys: the smaller node), the winner is appended and its consumers' counts of
// missing producers drop.
__global__ void __launch_bounds__(kDecodeWarps * 32)
decode_orders(DeviceGraph g, const float* __restrict__ keys, int P, int* __restrict__ orders_out) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int n = g.n;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p = blockIdx.x * kDecodeWarps + warp;
    if (p >= P) return;
    short* missing = reinterpret_cast<short*>(smem) + size_t(warp) * n;      // producers not yet placed; -1 once the node is placed
    float* key = reinterpret_cast<float*>(smem + round_up(size_t(kDecodeWarps) * n * 2, 16)) + size_t(warp) * n;
    for (int v = lane; v < n; v += 32) {
        missing[v] = short(g.pred_ptr[v + 1] - g.pred_ptr[v]);
        key[v] = keys[size_t(p) * n + v];
    }
    __syncwarp();
    for (int step = 0; step < n; ++step) {
        float bk = 0.0f;
        int bv = n;                                                          // n: no ready node seen
        for (int v = lane; v < n; v += 32) {
            if (missing[v] == 0) {
                const float kv = key[v];
                if (bv == n || kv > bk) { bk = kv; bv = v; }                 // v ascends within a lane: strict > keeps the smaller node
            }
        }
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) {
            const float ok = __shfl_xor_sync(0xffffffffu, bk, s);
            const int ov = __shfl_xor_sync(0xffffffffu, bv, s);
            if (ov != n && (bv == n || ok > bk || (ok == bk && ov < bv))) { bk = ok; bv = ov; }
        }
        if (bv == n) break;                                                  // cannot happen for an acyclic graph (checked at upload)
        if (lane == 0) {
            orders_out[size_t(p) * n + step] = bv;
            missing[bv] = -1;
        }
        for (int e = g.cons_ptr[bv] + lane; e < g.cons_ptr[bv + 1]; e += 32) missing[g.cons[e]] -= 1;    // consumers are distinct nodes
        __syncwarp();
    }
}

}  // namespace

struct mtpp_graph {
    DeviceGraph d;
    int device;
    int m;
    long long total_work;
    void* blob;
};

namespace {

std::mutex g_attr_lock;
bool g_attr_done[64] = {};

cudaError_t allow_slice_smem(int device) {
    std::lock_guard<std::mutex> guard(g_attr_lock);
    const bool tracked = device >= 0 && device < 64;
    if (tracked && g_attr_done[device]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(slice_orders<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSliceSmemLimit));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(slice_orders<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSliceSmemLimit));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(slice_orders<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSliceSmemLimit));
    if (e == cudaSuccess && tracked) g_attr_done[device] = true;
    return e;
}

}  // namespace

extern "C" {

int mtpp_graph_create(int n, int m, const int32_t* edges_host, const int64_t* work_host, const int64_t* sizeparam_host,
                      const int64_t* sizeout_host, mtpp_graph** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    if (n < 1 || n > MTPP_MAX_NODES || m < 0 || m > (1 << 22)) return BQ_ERR_SIZE;
    if ((m > 0 && !edges_host) || !work_host || !sizeparam_host || !sizeout_host) return BQ_ERR_NULL;
    constexpr long long kCap = 1LL << 40;
    long long tw = 0, tp = 0, ts = 0;
    for (int v = 0; v < n; ++v) {
        if (work_host[v] < 0 || sizeparam_host[v] < 0 || sizeout_host[v] < 0) return BQ_ERR_SIZE;
        if (work_host[v] >= kCap || sizeparam_host[v] >= kCap || sizeout_host[v] >= kCap) return BQ_ERR_SIZE;
        tw += work_host[v]; tp += sizeparam_host[v]; ts += sizeout_host[v];
        if (tw >= kCap || tp >= kCap || ts >= kCap) return BQ_ERR_SIZE;
    }
    // consumer lists without duplicates
    std::vector<std::vector<int>> cons(n), pred(n);
    for (int e = 0; e < m; ++e) {
        const int u = edges_host[2 * e], v = edges_host[2 * e + 1];
        if (u < 0 || u >= n || v < 0 || v >= n || u == v) return BQ_ERR_SIZE;
        bool seen = false;
        for (int c : cons[u]) seen = seen || (c == v);
        if (!seen) { cons[u].push_back(v); pred[v].push_back(u); }
    }
    // acyclic? (Kahn's count)
    {
        std::vector<int> missing(n), stack;
        for (int v = 0; v < n; ++v) { missing[v] = int(pred[v].size()); if (!missing[v]) stack.push_back(v); }
        int placed = 0;
        while (!stack.empty()) {
            const int v = stack.back(); stack.pop_back(); ++placed;
            for (int c : cons[v]) if (--missing[c] == 0) stack.push_back(c);
        }
        if (placed != n) return BQ_ERR_SIZE;
    }
    size_t edges = 0;
    for (int v = 0; v < n; ++v) edges += cons[v].size();
    // one blob: work | sizeparam | sizeout (int64) | pred_ptr | cons_ptr | pred | cons (int32)
    const size_t o_ptr = size_t(3) * n * 8, o_pred = o_ptr + size_t(2) * (n + 1) * 4, o_cons = o_pred + edges * 4, total = o_cons + edges * 4;
    std::vector<unsigned char> stage(total + 16, 0);
    long long* a64 = reinterpret_cast<long long*>(stage.data());
    for (int v = 0; v < n; ++v) { a64[v] = work_host[v]; a64[n + v] = sizeparam_host[v]; a64[2 * n + v] = sizeout_host[v]; }
    int* pp = reinterpret_cast<int*>(stage.data() + o_ptr);
    int* cp = pp + (n + 1);
    int* pl = reinterpret_cast<int*>(stage.data() + o_pred);
    int* cl = reinterpret_cast<int*>(stage.data() + o_cons);
    int np = 0, nc = 0;
    for (int v = 0; v < n; ++v) {
        pp[v] = np; cp[v] = nc;
        for (int u : pred[v]) pl[np++] = u;
        for (int c : cons[v]) cl[nc++] = c;
    }
    pp[n] = np; cp[n] = nc;
    mtpp_graph* g = new (std::nothrow) mtpp_graph();
    if (!g) return BQ_ERR_CUDA;
    cudaError_t e = cudaGetDevice(&g->device);
    if (e == cudaSuccess) e = cudaMalloc(&g->blob, total + 16);
    if (e == cudaSuccess) e = cudaMemcpy(g->blob, stage.data(), total, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        if (g->blob) cudaFree(g->blob);
        delete g;
        return cuda_fail(e);
    }
    const char* base = static_cast<const char*>(g->blob);
    g->d.n = n;
    g->d.work = reinterpret_cast<const long long*>(base);
    g->d.sizeparam = g->d.work + n;
    g->d.sizeout = g->d.sizeparam + n;
    g->d.pred_ptr = reinterpret_cast<const int*>(base + o_ptr);
    g->d.cons_ptr = g->d.pred_ptr + (n + 1);
    g->d.pred = reinterpret_cast<const int*>(base + o_pred);
    g->d.cons = reinterpret_cast<const int*>(base + o_cons);
    g->m = int(edges);
    g->total_work = tw;
    *out = g;
    return BQ_OK;
}

int mtpp_graph_free(mtpp_graph* g) {
    if (!g) return BQ_OK;
    const cudaError_t e = cudaFree(g->blob);
    delete g;
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int mtpp_decode_orders(const mtpp_graph* g, const float* keys, int P, int32_t* orders_out, void* cuda_stream) {
    if (!g) return BQ_ERR_NULL;
    if (P < 0 || P > (1 << 24)) return BQ_ERR_SIZE;
    if (P == 0) return BQ_OK;
    if (!keys || !orders_out) return BQ_ERR_NULL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != g->device) return BQ_ERR_CUDA;
    const size_t smem = round_up(size_t(kDecodeWarps) * g->d.n * 2, 16) + size_t(kDecodeWarps) * g->d.n * 4;
    const unsigned grid = unsigned((P + kDecodeWarps - 1) / kDecodeWarps);
    decode_orders<<<grid, kDecodeWarps * 32, smem, static_cast<cudaStream_t>(cuda_stream)>>>(g->d, keys, P, orders_out);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int mtpp_slice_orders(const mtpp_graph* g, const int32_t* orders, int P, int k, int64_t B, int64_t M, int64_t* cost_out, int32_t* blocks_out,
                      int32_t* cuts_out, int32_t* status_out, void* cuda_stream) {
    if (!g) return BQ_ERR_NULL;
    if (k < 1 || k > MTPP_MAX_BLOCKS) return BQ_ERR_BLOCK;
    if (P < 0 || P > (1 << 24) || B < 1 || M < 0 || M >= (1LL << 62)) return BQ_ERR_SIZE;
    if (g->total_work > 0 && B > (1LL << 62) / g->total_work) return BQ_ERR_SIZE;
    if (P == 0) return BQ_OK;
    if (!orders || !cost_out || !blocks_out || !cuts_out || !status_out) return BQ_ERR_NULL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != g->device) return BQ_ERR_CUDA;
    const int kmax = k < g->d.n ? k : g->d.n;
    // the graph rides in shared memory when it fits beside the programme's arrays
    int staged_edges = g->m > 0 ? g->m : 1;
    SliceLayout L = slice_layout(g->d.n, kmax, staged_edges);
    if (L.total > kSliceSmemLimit) {
        staged_edges = 0;
        L = slice_layout(g->d.n, kmax, 0);
    }
    cudaError_t e = cudaSuccess;
    if (L.total > 48 * 1024) e = allow_slice_smem(g->device);
    if (e != cudaSuccess) return cuda_fail(e);
    static_assert(MTPP_MAX_NODES <= 4 * kSliceThreads, "the widest instance owns four first positions per thread");
    auto* kernel = g->d.n <= kSliceThreads ? slice_orders<1> : g->d.n <= 2 * kSliceThreads ? slice_orders<2> : slice_orders<4>;
    kernel<<<unsigned(P), kSliceThreads, L.total, static_cast<cudaStream_t>(cuda_stream)>>>(
        g->d, staged_edges, orders, k, static_cast<long long>(B), static_cast<long long>(M), reinterpret_cast<long long*>(cost_out), blocks_out, cuts_out, status_out);
    e = cudaGetLastError();
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

}  // extern "C"
