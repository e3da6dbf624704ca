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
// So a CTA keeps five running values per l (in the registers of the thread that owns l), two columns,
// the dp rows of every block count, and per order a record of each position's node and three
// numbers per producer edge: a few tens of kilobytes of shared memory, no global scratch.  The
// column of r + 1 is written in the pass that takes the minima over the column of r (warp kk - 1
// for block count kk), so a step costs one barrier.
#include "../../include/mtpp.h"
#include "bq_error.h"

#include <cuda_runtime.h>

#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

namespace {

constexpr int kDecodeWarps = 4;
constexpr size_t kSliceSmemLimit = 226 * 1024;         // dynamic part of the 227 KB one CTA may take; the kernel's static words fit in the rest

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

struct DeviceGraph {
    int n;
    int edges;                 // distinct (producer, consumer) pairs
    const int* pred_ptr;       // [n + 1]
    const int* pred;           // producers of each node
    const int* cons_ptr;       // [n + 1]
    const int* cons;           // consumers of each node
    const long long* work;
    const long long* sizeparam;
    const long long* sizeout;
};

__host__ __device__ inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Shared memory of slice_orders for (n, kmax) and costs of `cs` bytes (8, or 4 when every segment cost of the call fits a
// signed 32-bit word): 16-byte records first, then the cost arrays, then 32-bit, then 16-bit.
struct SliceLayout {
    size_t attr, f, dp, eso, pos, last, epos, order, ethr, epu, arg, total;
};
// `edges` > 0: the producer edges of the order, re-laid in the order's own sequence (see the kernel), sit in shared memory
// too; 0: graphs with too many edges to fit beside the programme's arrays look them up in global memory at every step.
// rows of F and of dp start on 16-byte boundaries and are read four (two) words at a time
__host__ __device__ inline size_t slice_fstride(int n) { return round_up(size_t(n) + 4, 4); }
__host__ __device__ inline size_t slice_dstride(int n) { return round_up(size_t(n) + 1, 4); }
__host__ __device__ inline SliceLayout slice_layout(int n, int kmax, int edges, int cs) {
    SliceLayout L;
    size_t o = 0;
    L.attr = o; o += size_t(4) * n * cs;                               // by position: work, sizeparam, sizeout, sizeout if it has consumers
    L.f = o;    o += size_t(2) * slice_fstride(n) * cs;                // F(l, r) of the current r and of the next one
    L.dp = o;   o += size_t(kmax) * slice_dstride(n) * cs;             // dp[kk - 1][r]
    L.eso = o;  o += round_up(size_t(edges) * cs, 16);                 // per edge: the producer's sizeout
    L.pos = o;  o += size_t(n) * 4;                                    // 1-based position of each node (0: not seen)
    L.last = o; o += size_t(n) * 4;                                    // position of each node's last consumer (0: none)
    L.epos = o; o += size_t(n + 1) * 4;                                // edges of position r: [epos[r - 1], epos[r])
    L.order = o; o += size_t(n) * 4;                                   // the order itself
    L.ethr = o; o += round_up(size_t(edges) * 2, 4);                   // per edge: max(producer's position, its latest consumer before r)
    L.epu = o;  o += round_up(size_t(edges) * 2, 4);                   // per edge: producer's position if r is its last consumer, else 0
    L.arg = o;  o += size_t(kmax) * (n + 1) * 2;                       // the cut that gave dp[kk - 1][r]
    L.total = (o + 15) / 16 * 16;
    return L;
}

// The smallest (value, position) pair of a warp.  64-bit values: three 32-bit reductions (the high words, the low words among
// the lanes that hold the smallest high word, the positions among the lanes that hold the smallest value); 32-bit values: two.
__device__ __forceinline__ void warp_min_pair(long long& best, int& where) {
    const unsigned hi = unsigned(static_cast<unsigned long long>(best) >> 32), lo = unsigned(static_cast<unsigned long long>(best));
    const unsigned mh = __reduce_min_sync(0xffffffffu, hi);
    const unsigned ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
    const unsigned mi = __reduce_min_sync(0xffffffffu, (hi == mh && lo == ml) ? unsigned(where) : 0x7fffffffu);
    best = static_cast<long long>((static_cast<unsigned long long>(mh) << 32) | ml);
    where = int(mi);
}
__device__ __forceinline__ void warp_min_pair(int& best, int& where) {              // values are non-negative
    const int m = __reduce_min_sync(0xffffffffu, best);
    where = int(__reduce_min_sync(0xffffffffu, best == m ? unsigned(where) : 0x7fffffffu));
    best = m;
}

template <class C> struct alignas(4 * sizeof(C)) NodeRecord { C work, param, out, gain; };
template <class C> struct CostVec;                                   // 16 bytes of cost words
template <> struct CostVec<int> { using T = int4; static constexpr int N = 4; };
template <> struct CostVec<long long> { using T = longlong2; static constexpr int N = 2; };

// One CTA per order.  The n^2 segment costs are never tabulated: for a fixed right end r the costs F(l, r) of all first positions
// l form a column that follows from the column of r - 1 by adding the node at position r.  Per step of r: the owners of the
// first positions update their five running values and write the column, and warp kk - 1 takes
// dp[kk][r] = min over l of max(dp[kk - 1][l], F(l + 1, r)).  The column of r + 1 is written (into the other of two buffers)
// in the same pass that reads the column of r, so a step costs one barrier.
//
// What a step needs of the graph is prepared once per order, in the order's own sequence: a record of the node at position r
// (work, parameters, output, and the output again if it has consumers: they all come later), and for each producer u of that
// node the three things the update asks of an edge: u's output size; max(position of u, position of u's latest consumer before
// r), below which a first position l does not count u as an input any more; and u's position if r is u's last consumer (else 0),
// from which on l holds u inside and stops counting it as an output.
//
// C: the word costs are kept in.  int when the host has bounded every segment cost of the call below 2^31, long long otherwise.
template <int NT, int kOwned, class C, bool kEdgesInSmem>           // NT threads, kOwned first positions per thread: n <= kOwned * NT
__global__ void __launch_bounds__(NT)
slice_orders(DeviceGraph g, const int* __restrict__ orders, int k, C B, C M, long long* __restrict__ cost_out,
             int* __restrict__ blocks_out, int* __restrict__ cuts_out, int* __restrict__ status_out) {
    constexpr bool kNarrow = sizeof(C) == 4;
    constexpr C kInf = kNarrow ? C(0x7fffffff) : C(0x7fffffffffffffffLL);
    extern __shared__ __align__(16) unsigned char smem[];
    const int n = g.n;
    const int kmax = k < n ? k : n;
    const SliceLayout L = slice_layout(n, kmax, kEdgesInSmem ? g.edges : 0, int(sizeof(C)));
    NodeRecord<C>* attr = reinterpret_cast<NodeRecord<C>*>(smem + L.attr);
    C* F = reinterpret_cast<C*>(smem + L.f);
    C* dp = reinterpret_cast<C*>(smem + L.dp);
    C* eso = reinterpret_cast<C*>(smem + L.eso);
    int* pos = reinterpret_cast<int*>(smem + L.pos);
    int* last = reinterpret_cast<int*>(smem + L.last);
    int* epos = reinterpret_cast<int*>(smem + L.epos);
    int* ord = reinterpret_cast<int*>(smem + L.order);
    unsigned short* ethr = reinterpret_cast<unsigned short*>(smem + L.ethr);
    unsigned short* epu = reinterpret_cast<unsigned short*>(smem + L.epu);
    unsigned short* arg = reinterpret_cast<unsigned short*>(smem + L.arg);
    __shared__ int bad;

    const int p = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = NT / 32;
    constexpr int V = CostVec<C>::N;
    using VecT = typename CostVec<C>::T;
    const int fs = int(slice_fstride(n)), ds = int(slice_dstride(n));
    const int* pi = orders + size_t(p) * n;

    // positions, and the check that the row is a topological order of this graph
    if (tid == 0) bad = 0;
    for (int i = tid; i < n; i += NT) { pos[i] = 0; ord[i] = pi[i]; }
    __syncthreads();
    for (int i = tid; i < n; i += NT) {
        const int v = ord[i];
        if (v < 0 || v >= n) bad = 1;
        else if (atomicExch(&pos[v], i + 1) != 0) bad = 1;          // a node listed twice (so another one is missing)
    }
    __syncthreads();
    if (!bad) {
        for (int v = tid; v < n; v += NT) {
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
        for (int j = tid; j < k; j += NT) cuts_out[size_t(p) * k + j] = 0;
        return;
    }

    // the node records by position, and how many producer edges each position has
    if (tid == 0) epos[0] = 0;
    if (tid < kmax) dp[size_t(tid) * ds] = kInf;                     // no block holds the first 0 nodes: the vector reads below may start there
    for (int i = tid; i < n; i += NT) {
        const int v = ord[i];
        const C so = C(g.sizeout[v]);
        attr[i] = NodeRecord<C>{C(g.work[v]), C(g.sizeparam[v]), so, last[v] != 0 ? so : C(0)};
        epos[i + 1] = g.pred_ptr[v + 1] - g.pred_ptr[v];
    }
    __syncthreads();
    if (warp == 0) {                                                 // running sum of the counts: a chunk per lane, then across the lanes
        const int chunk = (n + 31) / 32, lo = 1 + lane * chunk, hi = (lo + chunk <= n + 1) ? lo + chunk : n + 1;
        int sum = 0;
        for (int i = lo; i < hi; ++i) sum += epos[i];
        int incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        int run = incl - sum;
        for (int i = lo; i < hi; ++i) { run += epos[i]; epos[i] = run; }
    }
    __syncthreads();
    // what the update asks of the edge u -> (node at position r)
    struct EdgeInfo { int thr, pu; C so; };
    auto edge_info = [&](int u, int r) -> EdgeInfo {
        const int pu = pos[u];
        int pc = 0;                                                  // u's latest consumer before r
        for (int e = g.cons_ptr[u]; e < g.cons_ptr[u + 1]; ++e) {
            const int q = pos[g.cons[e]];
            if (q < r && q > pc) pc = q;
        }
        return EdgeInfo{pu > pc ? pu : pc, last[u] == r ? pu : 0, C(g.sizeout[u])};
    };
    if constexpr (kEdgesInSmem) {
        for (int i = tid; i < n; i += NT) {
            const int v = ord[i];
            const int from = g.pred_ptr[v], at = epos[i], deg = epos[i + 1] - at;
            for (int j = 0; j < deg; ++j) {
                const EdgeInfo ei = edge_info(g.pred[from + j], i + 1);
                ethr[at + j] = static_cast<unsigned short>(ei.thr);
                epu[at + j] = static_cast<unsigned short>(ei.pu);
                eso[at + j] = ei.so;
            }
        }
        __syncthreads();
    }

    C cw[kOwned], cp[kOwned], ck[kOwned], ci[kOwned], co[kOwned];
#pragma unroll
    for (int j = 0; j < kOwned; ++j) { cw[j] = 0; cp[j] = 0; ck[j] = 0; ci[j] = 0; co[j] = 0; }
    // the column of r into Fw: thread t owns the first positions l = t + 1, t + 1 + NT, ... and keeps their five running values in registers
    auto column = [&](int r, C* __restrict__ Fw) {
        const NodeRecord<C> node = attr[r - 1];
        const int pb = epos[r - 1], pe = epos[r];
        const int from = kEdgesInSmem ? 0 : g.pred_ptr[ord[r - 1]];
#pragma unroll
        for (int j = 0; j < kOwned; ++j) {
            const int l = tid + 1 + j * NT;
            if (l > r) {
                if (l < r + V) Fw[l - 1] = kInf;                     // what a vector read of the column's end takes in beside it
                continue;
            }
            if (l == r) { cw[j] = 0; cp[j] = 0; ck[j] = 0; ci[j] = 0; co[j] = 0; }
            cw[j] += node.work;
            cp[j] += node.param;
            ck[j] = node.out > ck[j] ? node.out : ck[j];
            co[j] += node.gain;
            for (int e = pb; e < pe; ++e) {
                int thr, pu;
                C so_u;
                if constexpr (kEdgesInSmem) {
                    thr = ethr[e]; pu = epu[e]; so_u = eso[e];
                } else {
                    const EdgeInfo ei = edge_info(g.pred[from + e - pb], r);
                    thr = ei.thr; pu = ei.pu; so_u = ei.so;
                }
                if (l > thr) ci[j] += so_u;                          // u lies before l and nothing in l..r-1 read it
                if (pu >= l) co[j] -= so_u;                          // u is inside and this was its last consumer
            }
            const C excess = cp[j] + ck[j] - M;
            Fw[l - 1] = ci[j] + B * cw[j] + (excess > 0 ? excess : C(0)) + ck[j] + co[j];
        }
    };
    column(1, F + fs);                                               // the column of r sits in F + (r & 1) * fs
    __syncthreads();
    for (int r = 1; r <= n; ++r) {
        const C* __restrict__ Fr = F + (r & 1) * fs;
        // dp[kk][r] = min over l of max(dp[kk - 1][l], F(l + 1, r)); the earlier l on equal values
        for (int kk = warp + 1; kk <= kmax; kk += kWarps) {
            C best = kInf;
            int where = 0;
            if (kk == 1) {
                best = Fr[0];
            } else if (r >= kk) {
                // 16 bytes of each row per lane and trip.  Entries before l = kk - 1 hold "no such slicing" in the row below, entries
                // from l = r on hold it in the column: they never win.
                const C* below = dp + (kk - 2) * ds;
                for (int base = ((kk - 1) & ~(V - 1)) + lane * V; base < r; base += 32 * V) {
                    C a[V], b[V];
                    *reinterpret_cast<VecT*>(a) = *reinterpret_cast<const VecT*>(below + base);
                    *reinterpret_cast<VecT*>(b) = *reinterpret_cast<const VecT*>(Fr + base);
#pragma unroll
                    for (int i = 0; i < V; ++i) {
                        const C cand = a[i] > b[i] ? a[i] : b[i];
                        if (cand < best) { best = cand; where = base + i; }     // l ascends within a lane: strict < keeps the earlier one
                    }
                }
                warp_min_pair(best, where);
            }
            if (lane == 0) {
                dp[(kk - 1) * ds + r] = best;
                arg[(kk - 1) * (n + 1) + r] = static_cast<unsigned short>(where);
            }
        }
        if (r < n) column(r + 1, F + ((r + 1) & 1) * fs);            // the other buffer: nobody reads it before the barrier
        __syncthreads();
    }

    if (tid == 0) {
        int best_k = 1;
        for (int kk = 2; kk <= kmax; ++kk)
            if (dp[size_t(kk - 1) * ds + n] < dp[size_t(best_k - 1) * ds + n]) best_k = kk;
        cost_out[p] = static_cast<long long>(dp[size_t(best_k - 1) * ds + n]);
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

// Shared memory of decode_orders: per warp the counts of missing producers, the keys as ordered integers and the ready mask
// (a bit per node, word w owned by lane w); per CTA the consumer lists when `staged_edges` > 0.
struct DecodeLayout {
    size_t ukey, ready, missing, cptr, cons, total;
};
__host__ __device__ inline DecodeLayout decode_layout(int n, int staged_edges) {
    DecodeLayout L;
    size_t o = 0;
    L.ukey = o;    o += size_t(kDecodeWarps) * n * 4;
    L.ready = o;   o += size_t(kDecodeWarps) * 32 * 4;
    L.cptr = o;    o += staged_edges > 0 ? size_t(n + 1) * 4 : 0;
    L.cons = o;    o += staged_edges > 0 ? size_t(staged_edges) * 4 : 0;
    L.missing = o; o += size_t(kDecodeWarps) * n * 2;
    L.total = round_up(o, 16);
    return L;
}
constexpr int kDecodeStagedEdgesMax = 4096;                         // keeps the CTA within 48 KB at n = 1024

// One warp per key vector.  Ready nodes are a bit mask (at most 32 words: one per lane), so a step looks only at the nodes
// that are ready, not at all n: each lane walks the set bits of its word for its best key (equal keys: the smaller node),
// two warp reductions pick the winner (the largest key, then the smallest node that has it), the winner is appended, its bit
// cleared, and its consumers' counts of missing producers drop; a count that reaches zero sets the consumer's bit.
// Keys are compared as integers: k + 0.0f (which turns -0.0 into +0.0) mapped so that the order of finite floats is the
// order of unsigned words; no finite key maps to 0, which stands for "no ready node here".
__global__ void __launch_bounds__(kDecodeWarps * 32)
decode_orders(DeviceGraph g, int staged_edges, const float* __restrict__ keys, int P, int* __restrict__ orders_out) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int n = g.n;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p = blockIdx.x * kDecodeWarps + warp;
    const DecodeLayout L = decode_layout(n, staged_edges);
    unsigned* ukey = reinterpret_cast<unsigned*>(smem + L.ukey) + size_t(warp) * n;
    unsigned* ready = reinterpret_cast<unsigned*>(smem + L.ready) + warp * 32;
    short* missing = reinterpret_cast<short*>(smem + L.missing) + size_t(warp) * n;
    const int* cons_ptr = g.cons_ptr;
    const int* cons = g.cons;
    if (staged_edges > 0) {
        int* sp = reinterpret_cast<int*>(smem + L.cptr);
        int* sc = reinterpret_cast<int*>(smem + L.cons);
        for (int i = threadIdx.x; i <= n; i += kDecodeWarps * 32) sp[i] = g.cons_ptr[i];
        for (int i = threadIdx.x; i < staged_edges; i += kDecodeWarps * 32) sc[i] = g.cons[i];
        cons_ptr = sp;
        cons = sc;
        __syncthreads();
    }
    if (p >= P) return;
    const int words = (n + 31) / 32;
    for (int w = 0; w < words; ++w) {                                        // word w: nodes 32w .. 32w + 31, kept by lane w
        const int v = w * 32 + lane;
        int deg = 1;
        if (v < n) {
            deg = g.pred_ptr[v + 1] - g.pred_ptr[v];
            missing[v] = short(deg);
            const unsigned bits = __float_as_uint(keys[size_t(p) * n + v] + 0.0f);
            ukey[v] = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
        }
        const unsigned mask = __ballot_sync(0xffffffffu, deg == 0);
        if (lane == w) ready[lane] = mask;
    }
    if (lane >= words) ready[lane] = 0;
    __syncwarp();
    for (int step = 0; step < n; ++step) {
        unsigned w = ready[lane];
        unsigned bk = 0;
        int bv = 0x7fffffff;
        while (w) {
            const int v = lane * 32 + __ffs(int(w)) - 1;
            w &= w - 1;
            const unsigned kv = ukey[v];
            if (kv > bk) { bk = kv; bv = v; }                                // v ascends within a lane: strict > keeps the smaller node
        }
        const unsigned top = __reduce_max_sync(0xffffffffu, bk);
        if (top == 0) break;                                                 // no ready node: cannot happen for an acyclic graph (checked at upload)
        const int win = int(__reduce_min_sync(0xffffffffu, bk == top ? unsigned(bv) : 0x7fffffffu));
        if (lane == 0) {
            orders_out[size_t(p) * n + step] = win;
            atomicAnd(&ready[win >> 5], ~(1u << (win & 31)));
        }
        for (int e = cons_ptr[win] + lane; e < cons_ptr[win + 1]; e += 32) {  // consumers are distinct nodes
            const int c = cons[e];
            const short left = short(missing[c] - 1);
            missing[c] = left;
            if (left == 0) atomicOr(&ready[c >> 5], 1u << (c & 31));
        }
        __syncwarp();
    }
}

}  // namespace

struct mtpp_graph {
    DeviceGraph d;
    int device;
    int m;
    long long total_work, total_param, total_out, max_out;
    void* blob;
};

namespace {

std::mutex g_attr_lock;
bool g_attr_done[64] = {};

// The instances of slice_orders: (threads, first positions per thread) x cost word x where the edges are kept.  Small graphs take
// CTAs of four warps: what a step costs beside its arithmetic (the barrier, a warp's share of loop control) grows with the warps.
struct SliceShape { int threads, owned; };
inline SliceShape slice_shape(int n) {
    if (n <= 128) return {128, 1};
    if (n <= 256) return {128, 2};
    if (n <= 512) return {256, 2};
    return {256, 4};
}
template <int NT, int kOwned>
const void* slice_kernel_of(bool narrow, bool edges_in_smem) {
    if (narrow) return edges_in_smem ? reinterpret_cast<const void*>(&slice_orders<NT, kOwned, int, true>)
                                     : reinterpret_cast<const void*>(&slice_orders<NT, kOwned, int, false>);
    return edges_in_smem ? reinterpret_cast<const void*>(&slice_orders<NT, kOwned, long long, true>)
                         : reinterpret_cast<const void*>(&slice_orders<NT, kOwned, long long, false>);
}
const void* slice_kernel(SliceShape shape, bool narrow, bool edges_in_smem) {
    if (shape.threads == 128) return shape.owned == 1 ? slice_kernel_of<128, 1>(narrow, edges_in_smem) : slice_kernel_of<128, 2>(narrow, edges_in_smem);
    return shape.owned == 2 ? slice_kernel_of<256, 2>(narrow, edges_in_smem) : slice_kernel_of<256, 4>(narrow, edges_in_smem);
}
std::vector<const void*> slice_kernels() {
    std::vector<const void*> all;
    for (SliceShape shape : {SliceShape{128, 1}, SliceShape{128, 2}, SliceShape{256, 2}, SliceShape{256, 4}})
        for (bool narrow : {false, true})
            for (bool in_smem : {false, true}) all.push_back(slice_kernel(shape, narrow, in_smem));
    return all;
}

cudaError_t allow_slice_smem(int device) {
    std::lock_guard<std::mutex> guard(g_attr_lock);
    const bool tracked = device >= 0 && device < 64;
    if (tracked && g_attr_done[device]) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    for (const void* kernel : slice_kernels())
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSliceSmemLimit));
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
    long long tw = 0, tp = 0, ts = 0, mo = 0;
    for (int v = 0; v < n; ++v) {
        if (work_host[v] < 0 || sizeparam_host[v] < 0 || sizeout_host[v] < 0) return BQ_ERR_SIZE;
        if (work_host[v] >= kCap || sizeparam_host[v] >= kCap || sizeout_host[v] >= kCap) return BQ_ERR_SIZE;
        tw += work_host[v]; tp += sizeparam_host[v]; ts += sizeout_host[v];
        mo = sizeout_host[v] > mo ? sizeout_host[v] : mo;
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
    g->d.edges = int(edges);
    g->d.work = reinterpret_cast<const long long*>(base);
    g->d.sizeparam = g->d.work + n;
    g->d.sizeout = g->d.sizeparam + n;
    g->d.pred_ptr = reinterpret_cast<const int*>(base + o_ptr);
    g->d.cons_ptr = g->d.pred_ptr + (n + 1);
    g->d.pred = reinterpret_cast<const int*>(base + o_pred);
    g->d.cons = reinterpret_cast<const int*>(base + o_cons);
    g->m = int(edges);
    g->total_work = tw;
    g->total_param = tp;
    g->total_out = ts;
    g->max_out = mo;
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
    const int staged_edges = (g->d.edges > 0 && g->d.edges <= kDecodeStagedEdgesMax) ? g->d.edges : 0;     // larger lists stay in global memory
    const size_t smem = decode_layout(g->d.n, staged_edges).total;                                         // at most 45 KB
    const unsigned grid = unsigned((P + kDecodeWarps - 1) / kDecodeWarps);
    decode_orders<<<grid, kDecodeWarps * 32, smem, static_cast<cudaStream_t>(cuda_stream)>>>(g->d, staged_edges, keys, P, orders_out);
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
    // Every segment cost is at most in + out (disjoint sets of nodes: at most the sum of all outputs) + B * work + excess (at most
    // all parameters and one output) + peak (one output).  Below 2^31 the whole programme runs in 32-bit words.
    const long long cost_bound = g->total_out + 2 * g->max_out + g->total_param + B * g->total_work;     // no overflow: checked above
    const bool narrow = cost_bound < 0x7fffffffLL;
    const int cs = narrow ? 4 : 8;
    // the order's edges ride in shared memory when they fit beside the programme's arrays
    bool edges_in_smem = true;
    SliceLayout L = slice_layout(g->d.n, kmax, g->d.edges, cs);
    if (L.total > kSliceSmemLimit) {
        edges_in_smem = false;
        L = slice_layout(g->d.n, kmax, 0, cs);
    }
    if (L.total > kSliceSmemLimit) return BQ_ERR_SIZE;                // cannot happen within MTPP_MAX_NODES and MTPP_MAX_BLOCKS
    cudaError_t e = cudaSuccess;
    if (L.total > 48 * 1024) e = allow_slice_smem(g->device);
    if (e != cudaSuccess) return cuda_fail(e);
    static_assert(MTPP_MAX_NODES <= 4 * 256, "the widest instance owns four first positions per thread");
    const SliceShape shape = slice_shape(g->d.n);
    const void* kernel = slice_kernel(shape, narrow, edges_in_smem);
    long long* cost = reinterpret_cast<long long*>(cost_out);
    DeviceGraph d = g->d;
    long long B64 = B, M64 = M;
    int B32 = g->total_work > 0 ? int(B) : 0;                         // B * total_work < 2^31; without work the factor multiplies zeros
    int M32 = M < 0x7fffffffLL ? int(M) : 0x7fffffff;                 // parameters + peak stay below the bound: a larger M never shows
    void* args[] = {&d, &orders, &k, narrow ? static_cast<void*>(&B32) : static_cast<void*>(&B64),
                    narrow ? static_cast<void*>(&M32) : static_cast<void*>(&M64), &cost, &blocks_out, &cuts_out, &status_out};
    e = cudaLaunchKernel(kernel, dim3(unsigned(P)), dim3(unsigned(shape.threads)), args, L.total, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaGetLastError();
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

}  // extern "C"
