// mmd_api.cu -- the C ABI of the mixed matrix decomposition (see include/mmd.h): argument
// checks, the weight handle, tensor maps and the choice of kernel.
#include "../../include/mmd.h"
#include "bq_error.h"
#include "mmd_kernels.cuh"

#include <cstring>
#include <mutex>
#include <new>

namespace {

constexpr int kMaxK = 262144;
constexpr int kMaxFeatures = 1024;
constexpr size_t kWsAlign = 256;

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
bool is16(int dt) { return dt == BQ_F16 || dt == BQ_BF16; }

// cuTensorMapEncodeTiled through the runtime's entry-point lookup (no link against the driver library)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    // a function-local static is initialised once, under the language's own lock, however many threads arrive together
    static const EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        return EncodeTiledFn(nullptr);
    }();
    return fn;
}

// Per-device facts that the launchers look up on first use (shared-memory opt-ins, how many clusters run at once) are
// kept in small tables indexed by the device ordinal and written under this lock: two host threads may issue their
// first call at the same time.  mmd_decompose refuses devices beyond the tables, so an index is always in range.
constexpr int kMaxDevices = 64;
std::mutex g_cache_lock;

// Row-major [rows, cols] matrix of 1- or 2-byte elements, tiles of box_rows x 128 bytes, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * uint64_t(elem_bytes)};
    const cuuint32_t box[2] = {cuuint32_t(128 / elem_bytes), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = (elem_bytes == 1) ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16;
    return fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same matrix (K a multiple of 128, 1-byte elements) seen as (128 bytes, rows, K / 128): one load then brings
// `box_kblocks` K blocks of `box_rows` rows, laid out block after block, each with the 128-byte swizzle.
bool make_map_kblocks(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_kblocks) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 128 != 0) return false;
    const cuuint64_t dims[3] = {128, rows, cols / 128};
    const cuuint64_t strides[2] = {cols, 128};
    const cuuint32_t box[3] = {128, box_rows, box_kblocks};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DT>
cudaError_t launch_rowquant(const void* v, int R, int K, const int32_t* idx, int ko, int8_t* q, float* scale, void* side, int sm_count,
                            cudaStream_t stream, int* zero_words = nullptr, int n_zero_words = 0) {
    const size_t smem = round_up(size_t(K) / 8, 4);
    if (smem > 48 * 1024) return cudaErrorInvalidValue;          // K <= kMaxK keeps the mask within the default limit
    int grid = R;
    const int cap = sm_count * 16;
    if (grid > cap) grid = cap;
    // launched with programmatic stream serialization: the kernel waits (griddepcontrol.wait) for the kernels before it
    // before it touches global memory; behind a kernel that never signals its dependents this is an ordinary launch
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int side_cols = mmd_side_columns(ko);
    return cudaLaunchKernelEx(&cfg, mmdk::rowquant<DT>, v, R, K, idx, ko, side_cols, q, scale, side, zero_words, n_zero_words);
}

cudaError_t rowquant_any(int dt, const void* v, int R, int K, const int32_t* idx, int ko, int8_t* q, float* scale, void* side, int sm_count,
                         cudaStream_t stream, int* zero_words = nullptr, int n_zero_words = 0) {
    return dt == BQ_BF16 ? launch_rowquant<mmdk::kBF16>(v, R, K, idx, ko, q, scale, side, sm_count, stream, zero_words, n_zero_words)
                         : launch_rowquant<mmdk::kF16>(v, R, K, idx, ko, q, scale, side, sm_count, stream, zero_words, n_zero_words);
}

int check_features(const int32_t* idx_host, int ko, int K) {
    if (ko < 0 || ko > kMaxFeatures || ko >= K) return MMD_ERR_FEATURES;
    if (ko > 0 && !idx_host) return BQ_ERR_NULL;
    for (int j = 0; j < ko; ++j) {
        if (idx_host[j] < 0 || idx_host[j] >= K) return MMD_ERR_FEATURES;
        if (j > 0 && idx_host[j] <= idx_host[j - 1]) return MMD_ERR_FEATURES;
    }
    return BQ_OK;
}

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

}  // namespace

struct mmd_weights {
    int N, K, ko, side_cols, dtype, device, sm_count;
    void* blob;                  // q | scale | side | idx | status
    int8_t* q;
    float* scale;
    void* side;
    int32_t* idx;
    int* status;
    bool have_maps;
    CUtensorMap map_q[3], map_side[3];       // weight tiles of 256, 128 and 64 rows
    bool have_pair_map;                      // K a multiple of 128: the CTA-pair kernel's view of the codes
    CUtensorMap map_q_pair;                  // (128 bytes, rows, K / 128), boxes of 128 rows x 2 K blocks
};

namespace {

struct WsLayout { size_t q, scale, side, total; };

WsLayout ws_layout(const mmd_weights* w, int M) {
    WsLayout L;
    L.q = 0;
    L.scale = round_up(size_t(M) * w->K, kWsAlign);
    L.side = L.scale + round_up(size_t(M) * 4, kWsAlign);
    L.total = L.side + round_up(size_t(M) * w->side_cols * 2, kWsAlign);
    return L;
}

bool on_device(const mmd_weights* w) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == w->device;
}

int bn_slot(int bn) { return bn == 256 ? 0 : (bn == 128 ? 1 : 2); }

// Rows of the activation tiles the one-tile-per-CTA kernel loads: a decode step's few rows need only half a tile.
int activation_box_rows(int M) { return M <= 64 ? 64 : 128; }

template <int XDT, int YDT, int BN, int BM, int KPB>
cudaError_t launch_tc_bm(const mmd_weights* w, const CUtensorMap& mqx, const CUtensorMap& msx, const float* sx, void* y, int M, int split,
                         cudaStream_t stream, int n_tile_base = 0, int n_tile_count = -1) {
    using Cfg = mmdk::TcCfg<BN, BM, KPB>;
    static bool opted[kMaxDevices] = {};
    static int max_clusters[kMaxDevices][5] = {};
    if (w->device < 0 || w->device >= kMaxDevices) return cudaErrorInvalidDevice;
    const int d = w->device;
    std::lock_guard<std::mutex> guard(g_cache_lock);              // held to the end: the tables are read on the way to the launch
    if (!opted[d]) {
        const cudaError_t e = cudaFuncSetAttribute(mmdk::gemm_tc<XDT, YDT, BN, BM, KPB>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::kSmemBytes));
        if (e != cudaSuccess) return e;
        opted[d] = true;
    }
    int kblocks = (w->K + 127) / 128, sblocks = w->side_cols / 64;
    const int ksteps = (kblocks + KPB - 1) / KPB;
    const int slot = bn_slot(BN);
    CUtensorMap mqw = w->map_q[slot];
    if (KPB > 1 && !make_map_kblocks(&mqw, w->q, uint64_t(w->N), uint64_t(w->K), BN, KPB)) return cudaErrorInvalidValue;
    int* status = w->status;
    int Mv = M, Nv = w->N;
    const float* swv = w->scale;
    // the ranks' partial sums must fit into rank 0's ring
    if (split > 1 && size_t(split - 1) * BM * BN * 4 > size_t(Cfg::kStages) * Cfg::kStageBytes) split = 1;
    if (split > ksteps) split = ksteps;
    if (split > 4) split = 4;                                    // the largest cluster the exchange is written for (and the table below holds)
    if (split < 1) split = 1;
    cudaLaunchConfig_t cfg = {};
    if (n_tile_count < 0) n_tile_count = (w->N + BN - 1) / BN - n_tile_base;
    cfg.blockDim = dim3(mmdk::kTcThreads, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    // The split is there to put one CTA on every SM at the same time.  A cluster's CTAs must sit in one GPC, so fewer
    // clusters of 3 or 4 fit on the device than its SM count suggests; a split whose clusters would not all run at once
    // (a second, nearly empty wave) is lowered until they do.
    const long clusters = long((M + BM - 1) / BM) * n_tile_count;
    for (; split > 1; --split) {
        if (max_clusters[d][split] == 0) {
            cfg.gridDim = dim3(1, unsigned(w->sm_count / split), unsigned(split));
            attr[1].val.clusterDim.z = unsigned(split);
            cfg.attrs = &attr[1];
            cfg.numAttrs = 1;
            int n = 0;
            const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, mmdk::gemm_tc<XDT, YDT, BN, BM, KPB>, &cfg);
            if (e != cudaSuccess) return e;
            max_clusters[d][split] = n > 0 ? n : -1;
        }
        if (clusters <= max_clusters[d][split]) break;
    }
    cfg.gridDim = dim3(unsigned((M + BM - 1) / BM), unsigned(n_tile_count), unsigned(split));
    // The row kernel launched just before lets this kernel start early (its set-up and first weight loads overlap the row
    // kernel); the kernel itself waits for the row kernel's results before it touches them.
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].val.clusterDim.z = unsigned(split);
    cfg.attrs = attr;
    cfg.numAttrs = split > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, mmdk::gemm_tc<XDT, YDT, BN, BM, KPB>, mqx, mqw, sblocks ? msx : mqx,
                              sblocks ? w->map_side[slot] : w->map_q[slot], sx, swv, y, Mv, Nv, kblocks, sblocks, n_tile_base, status);
}

// At most 64 activation rows: 64-row MMAs and 64-row activation boxes (the host's maps are made to match).
template <int XDT, int YDT, int BN>
cudaError_t launch_tc(const mmd_weights* w, const CUtensorMap& mqx, const CUtensorMap& msx, const float* sx, void* y, int M, int split,
                      cudaStream_t stream) {
    return activation_box_rows(M) == 64 ? launch_tc_bm<XDT, YDT, BN, 64, 1>(w, mqx, msx, sx, y, M, split, stream)
                                        : launch_tc_bm<XDT, YDT, BN, 128, 1>(w, mqx, msx, sx, y, M, split, stream);
}

// 128-column tiles with K a multiple of 128: two K blocks per load (decode-size calls and mid-size products).  `mqx2` is
// the activations' three-dimensional map with boxes of activation_box_rows(M) rows x 2 K blocks.
template <int XDT, int YDT>
cudaError_t launch_tc_decode(const mmd_weights* w, const CUtensorMap& mqx2, const CUtensorMap& msx, const float* sx, void* y, int M, int split,
                             cudaStream_t stream, int n_tile_base = 0, int n_tile_count = -1) {
    return activation_box_rows(M) == 64 ? launch_tc_bm<XDT, YDT, 128, 64, 2>(w, mqx2, msx, sx, y, M, split, stream, n_tile_base, n_tile_count)
                                        : launch_tc_bm<XDT, YDT, 128, 128, 2>(w, mqx2, msx, sx, y, M, split, stream, n_tile_base, n_tile_count);
}

template <int XDT, int YDT>
cudaError_t launch_tcp(const mmd_weights* w, const CUtensorMap& mqx, const float* sx, const void* sidex, void* y, int M, cudaStream_t stream) {
    static bool opted[kMaxDevices] = {};
    if (w->device < 0 || w->device >= kMaxDevices) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> guard(g_cache_lock);
        if (!opted[w->device]) {
            const cudaError_t e = cudaFuncSetAttribute(mmdk::gemm_tcp<XDT, YDT>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(mmdk::kTcpSmemBytes));
            if (e != cudaSuccess) return e;
            opted[w->device] = true;
        }
    }
    const int mtiles = (M + 127) / 128, ntiles = (w->N + mmdk::kTcpBN - 1) / mmdk::kTcpBN;
    const long total = long(mtiles) * ntiles;
    const unsigned grid = unsigned(total < w->sm_count ? total : w->sm_count);
    mmdk::gemm_tcp<XDT, YDT><<<grid, mmdk::kTcThreads, mmdk::kTcpSmemBytes, stream>>>(
        mqx, w->map_q[0], sx, w->scale, sidex, w->side, w->side_cols, w->ko, y, M, w->N, (w->K + 127) / 128, mtiles, ntiles, w->status);
    return cudaGetLastError();
}

template <int XDT, int YDT>
cudaError_t launch_tc2(const mmd_weights* w, const CUtensorMap& mqx, const float* sx, const void* sidex, void* y, int M, cudaStream_t stream) {
    static bool opted[kMaxDevices] = {};
    static int max_pairs[kMaxDevices] = {};
    if (w->device < 0 || w->device >= kMaxDevices) return cudaErrorInvalidDevice;
    const int d = w->device;
    std::unique_lock<std::mutex> guard(g_cache_lock);
    if (!opted[d]) {
        cudaError_t e = cudaFuncSetAttribute(mmdk::gemm_tc2<XDT, YDT>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(mmdk::kPairSmemBytes));
        if (e != cudaSuccess) return e;
        // how many CTA pairs the device runs at once: the persistent grid must not exceed it
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(unsigned(w->sm_count & ~1), 1, 1);
        cfg.blockDim = dim3(mmdk::kTcThreads, 1, 1);
        cfg.dynamicSmemBytes = mmdk::kPairSmemBytes;
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, mmdk::gemm_tc2<XDT, YDT>, &cfg);
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorInvalidConfiguration;
        max_pairs[d] = n;
        opted[d] = true;
    }
    const int pairs_at_once = max_pairs[d];
    guard.unlock();
    const int mpairs = (M + 255) / 256, ntiles = (w->N + mmdk::kTcpBN - 1) / mmdk::kTcpBN;
    const long total = long(mpairs) * ntiles;
    const unsigned pairs = unsigned(total < pairs_at_once ? total : pairs_at_once);
    mmdk::gemm_tc2<XDT, YDT><<<2 * pairs, mmdk::kTcThreads, mmdk::kPairSmemBytes, stream>>>(
        mqx, w->map_q_pair, sx, w->scale, sidex, w->side, w->side_cols, w->ko, y, M, w->N, (w->K + 127) / 128, mpairs, ntiles, w->status);
    return cudaGetLastError();
}

// One row of tiles (a decode step of at most 64 rows) with the K steps of all tiles dealt out over one CTA per SM: the
// shape must have fewer 128-column tiles than SMs (so that a CTA's share touches at most two tiles) and the caller's
// workspace must have room, behind the decomposed activations, for the tiles' counters and partial sums.
struct SkPlan {
    bool ok;
    int n_tiles, grid, maxparts;
    size_t counters, acc, side, total;                     // offsets behind the base workspace, and the extra bytes
};

SkPlan sk_plan(const mmd_weights* w, int M) {
    SkPlan p = {};
    if (!w->have_maps || !w->have_pair_map || M < 1 || M > 64 || w->N < 1024 || w->N % 8 != 0) return p;
    p.n_tiles = (w->N + 127) / 128;
    if (p.n_tiles >= w->sm_count) return p;
    const long long ksteps = ((w->K + 127) / 128 + 1) / 2, upt = ksteps + (w->side_cols > 0 ? 1 : 0);
    const long long total = (long long)p.n_tiles * upt;
    if (ksteps < 8) return p;                              // too few steps per tile to be worth sharing
    const long long G = total < w->sm_count ? total : w->sm_count;
    p.grid = int(G);
    for (int t = 0; t < p.n_tiles; ++t) {
        const long long ta = (long long)t * upt, tb = ta + upt;
        const int c_first = int(((ta + 1) * G + total - 1) / total) - 1, c_last = int((tb * G + total - 1) / total) - 1;
        if (c_last - c_first + 1 > p.maxparts) p.maxparts = c_last - c_first + 1;
    }
    const size_t tile_values = size_t(64) * 128;
    p.counters = 0;
    p.acc = round_up(size_t(p.n_tiles) * 4, kWsAlign);
    p.side = p.acc + round_up(size_t(p.n_tiles) * p.maxparts * tile_values * 4, kWsAlign);
    p.total = p.side + (w->side_cols > 0 ? round_up(size_t(p.n_tiles) * tile_values * 4, kWsAlign) : 0);
    p.ok = true;
    return p;
}

template <int XDT, int YDT>
cudaError_t launch_sk(const mmd_weights* w, const SkPlan& p, const int8_t* qx, const void* sidex, const float* sx, void* y, int M, char* extra,
                      cudaStream_t stream) {
    using Cfg = mmdk::TcCfg<mmdk::kSkBN, mmdk::kSkBM, mmdk::kSkKPB>;
    static bool opted[kMaxDevices] = {};
    if (w->device < 0 || w->device >= kMaxDevices) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> guard(g_cache_lock);
        if (!opted[w->device]) {
            const cudaError_t e = cudaFuncSetAttribute(mmdk::gemm_sk<XDT, YDT>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::kSmemBytes));
            if (e != cudaSuccess) return e;
            opted[w->device] = true;
        }
    }
    CUtensorMap mqx, mqw, msx;
    if (!make_map_kblocks(&mqx, qx, uint64_t(M), uint64_t(w->K), 64, mmdk::kSkKPB)) return cudaErrorInvalidValue;
    if (!make_map_kblocks(&mqw, w->q, uint64_t(w->N), uint64_t(w->K), mmdk::kSkBN, mmdk::kSkKPB)) return cudaErrorInvalidValue;
    if (w->side_cols > 0) {
        if (!make_map(&msx, sidex, 2, uint64_t(M), uint64_t(w->side_cols), 64)) return cudaErrorInvalidValue;
    } else {
        msx = mqx;
    }
    const int slot = bn_slot(mmdk::kSkBN);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(p.grid), 1, 1);
    cfg.blockDim = dim3(mmdk::kTcThreads, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // starts under the row kernel; waits for it before reading its results
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, mmdk::gemm_sk<XDT, YDT>, mqx, mqw, msx, w->side_cols > 0 ? w->map_side[slot] : w->map_q[slot], sx,
                              static_cast<const float*>(w->scale), y, M, w->N, (w->K + 127) / 128, w->side_cols / 64, p.n_tiles, p.maxparts,
                              reinterpret_cast<int*>(extra + p.counters), reinterpret_cast<int*>(extra + p.acc),
                              reinterpret_cast<float*>(extra + p.side), w->status);
}

// Large products with few critical features take the persistent kernels.
bool wants_persistent(const mmd_weights* w, int M) {
    // from about half a wave of 128 x 256 tiles on: below that the one-tile-per-CTA kernel's narrower tiles fill the SMs better.
    // One row of tiles (a decode step) is bound by the weight stream, not by the tensor cores: it stays with that kernel too.
    return w->ko <= mmdk::kTcpSide && w->N >= 256 && M > 128 && long((M + 127) / 128) * ((w->N + 255) / 256) >= w->sm_count / 2;
}

template <int XDT, int YDT>
cudaError_t launch_tc_bn(const mmd_weights* w, const CUtensorMap& mqx, const CUtensorMap& msx, const int8_t* qx, const float* sx, void* y, int M,
                         cudaStream_t stream) {
    // The widest tile has the highest arithmetic intensity; when it would leave SMs without a
    // tile (few rows, as in a decode step, where the weights are read once and the kernel is
    // bound by that stream) narrower tiles put more CTAs on the weight stream.
    const long mt = (M + 127) / 128;
    if (w->N >= 256 && mt * ((w->N + 255) / 256) >= w->sm_count) return launch_tc<XDT, YDT, 256>(w, mqx, msx, sx, y, M, 1, stream);
    if (w->N >= 128 && mt * ((w->N + 127) / 128) >= w->sm_count) {
        CUtensorMap mqx2;                                                        // K a multiple of 128: two K blocks per load
        if (w->have_pair_map && make_map_kblocks(&mqx2, qx, uint64_t(M), uint64_t(w->K), uint32_t(activation_box_rows(M)), 2)) {
            // One row of tiles that does not fill whole waves (a decode step through a wide layer): the whole waves run one
            // tile per CTA, and the tiles left over share their K steps among 2-4 CTAs each, so that the last wave also
            // keeps about one CTA per SM on the weight stream instead of running at full length on a few SMs.
            const long tiles = (w->N + 127) / 128;
            const long rest = tiles % w->sm_count;
            if (mt == 1 && rest > 0 && rest <= w->sm_count / 2) {
                int split = int(w->sm_count / rest);
                if (split > 4) split = 4;
                while (split > 1 && (w->K + 255) / 256 < 4 * split) --split;    // at least 4 steps per CTA
                if (split > 1) {
                    const cudaError_t e = launch_tc_decode<XDT, YDT>(w, mqx2, msx, sx, y, M, 1, stream, 0, int(tiles - rest));
                    if (e != cudaSuccess) return e;
                    return launch_tc_decode<XDT, YDT>(w, mqx2, msx, sx, y, M, split, stream, int(tiles - rest), int(rest));
                }
            }
            return launch_tc_decode<XDT, YDT>(w, mqx2, msx, sx, y, M, 1, stream);
        }
        return launch_tc<XDT, YDT, 128>(w, mqx, msx, sx, y, M, 1, stream);
    }
    // One row of tiles (a decode step) streams every weight once from DRAM, and an SM streams only as fast as the bytes it
    // keeps in flight.  128-row weight tiles hold the most per CTA; when they leave SMs idle, 2-4 CTAs share each tile's K
    // steps (clusters along z) so that about one CTA per SM is streaming.
    if (mt == 1 && w->N >= 1024) {
        const long tiles = (w->N + 127) / 128;
        int split = int(w->sm_count / tiles);
        if (split > 4) split = 4;
        if (split < 1) split = 1;
        if (w->have_pair_map) {                                                  // K a multiple of 128: two K blocks per load
            while (split > 1 && (w->K + 255) / 256 < 4 * split) --split;        // at least 4 steps per CTA
            CUtensorMap mqx2;
            if (make_map_kblocks(&mqx2, qx, uint64_t(M), uint64_t(w->K), uint32_t(activation_box_rows(M)), 2))
                return launch_tc_decode<XDT, YDT>(w, mqx2, msx, sx, y, M, split, stream);
        }
        while (split > 1 && (w->K + 127) / 128 < 8 * split) --split;            // at least 8 steps per CTA
        return launch_tc<XDT, YDT, 128>(w, mqx, msx, sx, y, M, split, stream);
    }
    return launch_tc<XDT, YDT, 64>(w, mqx, msx, sx, y, M, 1, stream);
}

template <int XDT, int YDT>
cudaError_t launch_general(const mmd_weights* w, const int8_t* qx, const float* sx, const void* sidex, void* y, int M, cudaStream_t stream) {
    const dim3 grid(unsigned((w->N + 63) / 64), unsigned((M + 63) / 64));
    mmdk::gemm_general<XDT, YDT><<<grid, 256, 0, stream>>>(qx, w->q, sx, w->scale, sidex, w->side, w->side_cols, y, M, w->N, w->K);
    return cudaGetLastError();
}

}  // namespace

extern "C" {

int mmd_side_columns(int n_features) {
    return n_features <= 0 ? 0 : (n_features + mmdk::kSidePad - 1) / mmdk::kSidePad * mmdk::kSidePad;
}

int mmd_select_features(const float* feature_absmax, int K, float tau, int32_t* idx_out, int* count_out) {
    if (!feature_absmax || !idx_out || !count_out) return BQ_ERR_NULL;
    if (K < 1) return BQ_ERR_SIZE;
    int c = 0;
    for (int k = 0; k < K; ++k)
        if (feature_absmax[k] >= tau) idx_out[c++] = k;
    *count_out = c;
    return BQ_OK;
}

int mmd_rowquant(const void* v, bq_dtype dt, int R, int K, const int32_t* idx, int n_features, int8_t* q_out, float* scale_out,
                 void* side_out, void* cuda_stream) {
    if (!is16(dt)) return BQ_ERR_DTYPE;
    if (R < 0 || K < 16 || K % 16 != 0 || K > kMaxK) return BQ_ERR_SIZE;
    if (n_features < 0 || n_features > kMaxFeatures || n_features >= K) return MMD_ERR_FEATURES;
    if (R == 0) return BQ_OK;
    if (!v || !q_out || !scale_out || (n_features > 0 && (!idx || !side_out))) return BQ_ERR_NULL;
    if (!aligned(v, 16) || !aligned(q_out, 16)) return BQ_ERR_SIZE;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = rowquant_any(dt, v, R, K, idx, n_features, q_out, scale_out, side_out, sms, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int mmd_decompose(const void* W, bq_dtype dt, int N, int K, const int32_t* idx_host, int n_features, void* cuda_stream, mmd_weights** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    if (!is16(dt)) return BQ_ERR_DTYPE;
    if (N < 1 || K < 16 || K % 16 != 0 || K > kMaxK) return BQ_ERR_SIZE;
    const int fc = check_features(idx_host, n_features, K);
    if (fc != BQ_OK) return fc;
    if (!W) return BQ_ERR_NULL;
    if (!aligned(W, 16)) return BQ_ERR_SIZE;
    mmd_weights* w = new (std::nothrow) mmd_weights();
    if (!w) return BQ_ERR_CUDA;
    w->N = N; w->K = K; w->ko = n_features; w->side_cols = mmd_side_columns(n_features); w->dtype = dt;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaGetDevice(&w->device);
    if (e == cudaSuccess && (w->device < 0 || w->device >= kMaxDevices)) e = cudaErrorInvalidDevice;     // beyond the per-device tables
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&w->sm_count, cudaDevAttrMultiProcessorCount, w->device);
    const size_t o_q = 0;
    const size_t o_scale = round_up(size_t(N) * K, kWsAlign);
    const size_t o_side = o_scale + round_up(size_t(N) * 4, kWsAlign);
    const size_t o_idx = o_side + round_up(size_t(N) * w->side_cols * 2, kWsAlign);
    const size_t o_status = o_idx + round_up(size_t(kMaxFeatures) * 4, kWsAlign);
    const size_t total = o_status + kWsAlign;
    if (e == cudaSuccess) e = cudaMalloc(&w->blob, total);
    if (e != cudaSuccess) { delete w; return cuda_fail(e); }
    char* base = static_cast<char*>(w->blob);
    w->q = reinterpret_cast<int8_t*>(base + o_q);
    w->scale = reinterpret_cast<float*>(base + o_scale);
    w->side = base + o_side;
    w->idx = reinterpret_cast<int32_t*>(base + o_idx);
    w->status = reinterpret_cast<int*>(base + o_status);
    e = cudaMemsetAsync(w->status, 0, sizeof(int), stream);
    // the feature list is copied from pageable host memory: the copy has left the host buffer when the call returns
    if (e == cudaSuccess && n_features > 0) e = cudaMemcpyAsync(w->idx, idx_host, size_t(n_features) * 4, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = rowquant_any(dt, W, N, K, w->idx, n_features, w->q, w->scale, w->side, w->sm_count, stream);
    if (e != cudaSuccess) { cudaFree(w->blob); delete w; return cuda_fail(e); }
    w->have_maps = true;
    w->have_pair_map = make_map_kblocks(&w->map_q_pair, w->q, uint64_t(N), uint64_t(K), 128, mmdk::kPairStepBlocks);
    const uint32_t boxes[3] = {256, 128, 64};
    for (int s = 0; s < 3; ++s) {
        w->have_maps = w->have_maps && make_map(&w->map_q[s], w->q, 1, uint64_t(N), uint64_t(K), boxes[s]);
        if (w->side_cols > 0) w->have_maps = w->have_maps && make_map(&w->map_side[s], w->side, 2, uint64_t(N), uint64_t(w->side_cols), boxes[s]);
    }
    *out = w;
    return BQ_OK;
}

int mmd_free(mmd_weights* w) {
    if (!w) return BQ_OK;
    const cudaError_t e = cudaFree(w->blob);
    delete w;
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int mmd_weights_view(const mmd_weights* w, const int8_t** q, const float** scale, const void** side, const int32_t** idx, int* N, int* K,
                     int* n_features, int* dtype) {
    if (!w) return BQ_ERR_NULL;
    if (q) *q = w->q;
    if (scale) *scale = w->scale;
    if (side) *side = w->side;
    if (idx) *idx = w->idx;
    if (N) *N = w->N;
    if (K) *K = w->K;
    if (n_features) *n_features = w->ko;
    if (dtype) *dtype = w->dtype;
    return BQ_OK;
}

int mmd_workspace_layout(const mmd_weights* w, int M, size_t* offsets3, size_t* total_bytes) {
    if (!w || !total_bytes) return BQ_ERR_NULL;
    if (M < 0) return BQ_ERR_SIZE;
    const WsLayout L = ws_layout(w, M);
    if (offsets3) { offsets3[0] = L.q; offsets3[1] = L.scale; offsets3[2] = L.side; }
    *total_bytes = L.total;
    return BQ_OK;
}

int mmd_workspace_bytes_streamk(const mmd_weights* w, int M, size_t* total_bytes) {
    if (!w || !total_bytes) return BQ_ERR_NULL;
    if (M < 0) return BQ_ERR_SIZE;
    const SkPlan p = sk_plan(w, M);
    *total_bytes = ws_layout(w, M).total + (p.ok ? p.total : 0);
    return BQ_OK;
}

int mmd_linear(const mmd_weights* w, const void* X, int M, void* Y, bq_dtype ydt, void* workspace, size_t workspace_bytes, int path,
               void* cuda_stream) {
    if (!w) return BQ_ERR_NULL;
    if (ydt != BQ_F32 && int(ydt) != w->dtype) return BQ_ERR_DTYPE;
    if (M < 0) return BQ_ERR_SIZE;
    if (path < MMD_PATH_AUTO || path > MMD_PATH_TENSOR_STREAMK) return MMD_ERR_PATH;
    if (M == 0) return BQ_OK;
    if (!X || !Y) return BQ_ERR_NULL;
    if (!aligned(X, 16)) return BQ_ERR_SIZE;
    const WsLayout L = ws_layout(w, M);
    if (!workspace || !aligned(workspace, kWsAlign) || workspace_bytes < L.total) return MMD_ERR_WORKSPACE;
    if (!on_device(w)) return BQ_ERR_CUDA;
    const bool tc_ok = w->have_maps && (w->N % 8 == 0) && aligned(Y, 16);
    if (path >= MMD_PATH_TENSOR && !tc_ok) return MMD_ERR_PATH;
    if (path == MMD_PATH_TENSOR_SOLO && !wants_persistent(w, M)) return MMD_ERR_PATH;
    const bool use_tc = (path >= MMD_PATH_TENSOR) || (path == MMD_PATH_AUTO && tc_ok);
    const bool persistent = use_tc && path != MMD_PATH_TENSOR_TILE && wants_persistent(w, M);
    const bool pairs = persistent && path != MMD_PATH_TENSOR_SOLO && w->have_pair_map;      // the pair kernel's loads need K % 128 == 0
    // a decode step over a layer with fewer tiles than SMs, on request: all tiles' K steps over one CTA per SM.  Not taken by
    // AUTO: as measured, handing partial sums over through global memory costs more than the even shares save.
    const SkPlan sk = (use_tc && !persistent && path == MMD_PATH_TENSOR_STREAMK) ? sk_plan(w, M) : SkPlan{};
    const bool stream_k = sk.ok && workspace_bytes >= L.total + sk.total;
    if (path == MMD_PATH_TENSOR_STREAMK && !stream_k) return sk.ok ? MMD_ERR_WORKSPACE : MMD_ERR_PATH;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    int8_t* qx = reinterpret_cast<int8_t*>(ws + L.q);
    float* sx = reinterpret_cast<float*>(ws + L.scale);
    void* sidex = ws + L.side;
    cudaError_t e = rowquant_any(w->dtype, X, M, w->K, w->idx, w->ko, qx, sx, sidex, w->sm_count, stream,
                                 stream_k ? reinterpret_cast<int*>(ws + L.total + sk.counters) : nullptr, stream_k ? sk.n_tiles : 0);
    if (e != cudaSuccess) return cuda_fail(e);

    const bool bf = (w->dtype == BQ_BF16), f32out = (ydt == BQ_F32);
    if (stream_k) {
        char* extra = ws + L.total;
        if (bf) e = f32out ? launch_sk<mmdk::kBF16, mmdk::kF32>(w, sk, qx, sidex, sx, Y, M, extra, stream) : launch_sk<mmdk::kBF16, mmdk::kBF16>(w, sk, qx, sidex, sx, Y, M, extra, stream);
        else e = f32out ? launch_sk<mmdk::kF16, mmdk::kF32>(w, sk, qx, sidex, sx, Y, M, extra, stream) : launch_sk<mmdk::kF16, mmdk::kF16>(w, sk, qx, sidex, sx, Y, M, extra, stream);
    } else if (pairs) {
        CUtensorMap mqx;
        if (!make_map_kblocks(&mqx, qx, uint64_t(M), uint64_t(w->K), 128, mmdk::kPairStepBlocks)) return MMD_ERR_PATH;
        if (bf) e = f32out ? launch_tc2<mmdk::kBF16, mmdk::kF32>(w, mqx, sx, sidex, Y, M, stream) : launch_tc2<mmdk::kBF16, mmdk::kBF16>(w, mqx, sx, sidex, Y, M, stream);
        else e = f32out ? launch_tc2<mmdk::kF16, mmdk::kF32>(w, mqx, sx, sidex, Y, M, stream) : launch_tc2<mmdk::kF16, mmdk::kF16>(w, mqx, sx, sidex, Y, M, stream);
    } else if (persistent) {
        CUtensorMap mqx;
        if (!make_map(&mqx, qx, 1, uint64_t(M), uint64_t(w->K), 128)) return MMD_ERR_PATH;
        if (bf) e = f32out ? launch_tcp<mmdk::kBF16, mmdk::kF32>(w, mqx, sx, sidex, Y, M, stream) : launch_tcp<mmdk::kBF16, mmdk::kBF16>(w, mqx, sx, sidex, Y, M, stream);
        else e = f32out ? launch_tcp<mmdk::kF16, mmdk::kF32>(w, mqx, sx, sidex, Y, M, stream) : launch_tcp<mmdk::kF16, mmdk::kF16>(w, mqx, sx, sidex, Y, M, stream);
    } else if (use_tc) {
        CUtensorMap mqx, msx;
        const uint32_t arows = uint32_t(activation_box_rows(M));
        if (!make_map(&mqx, qx, 1, uint64_t(M), uint64_t(w->K), arows)) return MMD_ERR_PATH;
        if (w->side_cols > 0 && !make_map(&msx, sidex, 2, uint64_t(M), uint64_t(w->side_cols), arows)) return MMD_ERR_PATH;
        if (w->side_cols == 0) msx = mqx;
        if (bf) e = f32out ? launch_tc_bn<mmdk::kBF16, mmdk::kF32>(w, mqx, msx, qx, sx, Y, M, stream) : launch_tc_bn<mmdk::kBF16, mmdk::kBF16>(w, mqx, msx, qx, sx, Y, M, stream);
        else e = f32out ? launch_tc_bn<mmdk::kF16, mmdk::kF32>(w, mqx, msx, qx, sx, Y, M, stream) : launch_tc_bn<mmdk::kF16, mmdk::kF16>(w, mqx, msx, qx, sx, Y, M, stream);
    } else {
        if (bf) e = f32out ? launch_general<mmdk::kBF16, mmdk::kF32>(w, qx, sx, sidex, Y, M, stream) : launch_general<mmdk::kBF16, mmdk::kBF16>(w, qx, sx, sidex, Y, M, stream);
        else e = f32out ? launch_general<mmdk::kF16, mmdk::kF32>(w, qx, sx, sidex, Y, M, stream) : launch_general<mmdk::kF16, mmdk::kF16>(w, qx, sx, sidex, Y, M, stream);
    }
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int mmd_selftest_bounded_wait(const mmd_weights* w, unsigned limit_us, int* threads_left_out, void* cuda_stream) {
    if (!w || !threads_left_out) return BQ_ERR_NULL;
    if (limit_us < 1 || limit_us > 100000) return BQ_ERR_SIZE;              // 1 us .. 0.1 s: this wait is meant to run out
    if (!on_device(w)) return BQ_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int khz = 0;
    cudaError_t e = cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, w->device);
    if (e != cudaSuccess) return cuda_fail(e);
    const long long cycles = (long long)limit_us * (khz > 0 ? khz : 1000000) / 1000;
    // the counter lives in the handle's spare status space (the word after the status)
    int* left = w->status + 1;
    e = cudaMemsetAsync(left, 0, sizeof(int), stream);
    if (e != cudaSuccess) return cuda_fail(e);
    mmdk::wait_selftest<<<1, mmdk::kTcThreads, 0, stream>>>(w->status, MMD_SELFTEST_CODE, cycles, left);
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(threads_left_out, left, sizeof(int), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int mmd_kernel_status(const mmd_weights* w, int* status_out) {
    if (!w || !status_out) return BQ_ERR_NULL;
    if (!on_device(w)) return BQ_ERR_CUDA;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(status_out, w->status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && *status_out != 0) e = cudaMemset(w->status, 0, sizeof(int));
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

}  // extern "C"
