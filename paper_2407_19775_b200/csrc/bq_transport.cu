// bq_transport.cu -- the boundary transport of include/bq_transport.h: a mailbox in the receiving
// shard's memory, filled piece by piece by the sending shard's quantize kernel (its stores cross
// the link) and drained by the receiving shard's dequantize kernel, ordered by two events per slot.
// This file owns memory, events and ordering; the arithmetic is in the kernels behind bq_quantize
// and bq_dequantize.
#include "../../include/bq_transport.h"
#include "bq_error.h"

#include <cuda_runtime.h>
#include <unistd.h>

#include <cstdio>
#include <cstring>
#include <new>

namespace {

constexpr int kMaxSlots = 8;
constexpr uint32_t kMagic = 0x62717831u;          // "bqx1"

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
bool known_dtype(int dt) { return dt == BQ_F32 || dt == BQ_F16 || dt == BQ_BF16; }

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}
int fail_text(const char* text) {
    bql::set_last_cuda_error(text);
    return BQ_ERR_CUDA;
}

// One slot: codes (chunk bytes, rounded up to 256) followed by its absmax floats.
struct Geometry {
    size_t chunk;
    int min_block, slots;
    size_t codes_bytes, absmax_bytes, slot_bytes;
};

bool make_geometry(size_t chunk, int min_block, int slots, Geometry* g) {
    if (chunk == 0 || chunk >= (size_t(1) << 34) || min_block < 1 || size_t(min_block) > chunk || slots < 2 || slots > kMaxSlots) return false;
    g->chunk = chunk;
    g->min_block = min_block;
    g->slots = slots;
    g->codes_bytes = round_up(chunk, 256);
    g->absmax_bytes = round_up((chunk / size_t(min_block) + 1) * 4, 256);
    g->slot_bytes = g->codes_bytes + g->absmax_bytes;
    return true;
}

// What bqx_rx_export writes and bqx_tx_open reads.
struct Description {
    uint32_t magic;
    int32_t pid, device, slots, min_block;
    uint64_t chunk;
    uint64_t mailbox;                       // the pointer, valid in the owning process
    uint64_t filled[kMaxSlots], drained[kMaxSlots];     // the events, valid in the owning process
    cudaIpcMemHandle_t mem;
    cudaIpcEventHandle_t filled_ipc[kMaxSlots], drained_ipc[kMaxSlots];
    int32_t have_ipc;
};
static_assert(sizeof(Description) <= BQX_EXPORT_BYTES, "the description fits the export buffer");

#define BQ_TRY(expr)                                   \
    do {                                               \
        const cudaError_t e_ = (expr);                 \
        if (e_ != cudaSuccess) return cuda_fail(e_);   \
    } while (0)

}  // namespace

struct bqx_rx {
    const bq_codebook* cb;
    int device;
    Geometry g;
    char* mailbox;
    cudaEvent_t filled[kMaxSlots], drained[kMaxSlots];
};

struct bqx_tx {
    const bq_codebook* cb;
    int device, rx_device;
    Geometry g;
    int mode;
    bool remote_process;                   // mailbox and events were opened through IPC handles
    char* mailbox;                         // the receiver's mailbox as this process / device sees it
    char* staging;                         // BQX_COPY: slots * slot_bytes on the sender
    cudaEvent_t filled[kMaxSlots], drained[kMaxSlots];
    bool used[kMaxSlots];                  // the slot has been filled before (in this or an earlier tensor): wait for its drain
};

extern "C" {

size_t bqx_mailbox_bytes(size_t chunk_elems, int min_block, int slots) {
    Geometry g;
    return make_geometry(chunk_elems, min_block, slots, &g) ? g.slot_bytes * size_t(slots) : 0;
}

size_t bqx_payload_bytes(size_t n, int block) { return block < 1 ? 0 : n + 4 * ((n + size_t(block) - 1) / size_t(block)); }

int bqx_plan(size_t n, int block, size_t chunk_elems, int slots, size_t p, size_t* pieces, int* slot, size_t* first, size_t* count) {
    if (block < 1 || size_t(block) > chunk_elems) return BQ_ERR_BLOCK;
    if (slots < 1) return BQ_ERR_SIZE;
    const size_t piece = (chunk_elems / size_t(block)) * size_t(block);
    const size_t np = (n + piece - 1) / piece;
    if (pieces) *pieces = np;
    if (p >= np) return BQ_ERR_SIZE;
    if (slot) *slot = int(p % size_t(slots));
    if (first) *first = p * piece;
    if (count) *count = (n - p * piece < piece) ? n - p * piece : piece;
    return BQ_OK;
}

int bqx_rx_create(const bq_codebook* cb, size_t chunk_elems, int min_block, int slots, bqx_rx** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    if (!cb) return BQ_ERR_CODEBOOK;
    Geometry g;
    if (min_block < 1 || (chunk_elems > 0 && size_t(min_block) > chunk_elems)) return BQ_ERR_BLOCK;
    if (!make_geometry(chunk_elems, min_block, slots, &g)) return BQ_ERR_SIZE;
    bqx_rx* rx = new (std::nothrow) bqx_rx();
    if (!rx) return BQ_ERR_CUDA;
    rx->cb = cb;
    rx->g = g;
    cudaError_t e = cudaGetDevice(&rx->device);
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&rx->mailbox), g.slot_bytes * size_t(slots));
    for (int s = 0; s < slots && e == cudaSuccess; ++s) {
        e = cudaEventCreateWithFlags(&rx->filled[s], cudaEventDisableTiming | cudaEventInterprocess);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&rx->drained[s], cudaEventDisableTiming | cudaEventInterprocess);
    }
    if (e != cudaSuccess) {
        bqx_rx_destroy(rx);
        return cuda_fail(e);
    }
    *out = rx;
    return BQ_OK;
}

int bqx_rx_destroy(bqx_rx* rx) {
    if (!rx) return BQ_OK;
    for (int s = 0; s < kMaxSlots; ++s) {
        if (rx->filled[s]) cudaEventDestroy(rx->filled[s]);
        if (rx->drained[s]) cudaEventDestroy(rx->drained[s]);
    }
    cudaError_t e = cudaSuccess;
    if (rx->mailbox) e = cudaFree(rx->mailbox);
    delete rx;
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bqx_rx_export(const bqx_rx* rx, void* out) {
    if (!rx || !out) return BQ_ERR_NULL;
    Description d;
    std::memset(&d, 0, sizeof(d));
    d.magic = kMagic;
    d.pid = int32_t(getpid());
    d.device = rx->device;
    d.slots = rx->g.slots;
    d.min_block = rx->g.min_block;
    d.chunk = rx->g.chunk;
    d.mailbox = uint64_t(reinterpret_cast<uintptr_t>(rx->mailbox));
    // IPC handles serve a sender in another process; where the platform refuses them the
    // description still serves a sender in this process
    d.have_ipc = (cudaIpcGetMemHandle(&d.mem, rx->mailbox) == cudaSuccess) ? 1 : 0;
    for (int s = 0; s < rx->g.slots; ++s) {
        d.filled[s] = uint64_t(reinterpret_cast<uintptr_t>(rx->filled[s]));
        d.drained[s] = uint64_t(reinterpret_cast<uintptr_t>(rx->drained[s]));
        if (d.have_ipc && (cudaIpcGetEventHandle(&d.filled_ipc[s], rx->filled[s]) != cudaSuccess ||
                           cudaIpcGetEventHandle(&d.drained_ipc[s], rx->drained[s]) != cudaSuccess))
            d.have_ipc = 0;
    }
    if (!d.have_ipc) (void)cudaGetLastError();       // a refused handle leaves no error behind
    std::memset(out, 0, BQX_EXPORT_BYTES);
    std::memcpy(out, &d, sizeof(d));
    return BQ_OK;
}

int bqx_tx_open(const bq_codebook* cb, const void* description, int mode, bqx_tx** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (!description) return BQ_ERR_NULL;
    if (mode != BQX_STORE && mode != BQX_COPY) return BQ_ERR_SIZE;
    Description d;
    std::memcpy(&d, description, sizeof(d));
    Geometry g;
    if (d.magic != kMagic || !make_geometry(size_t(d.chunk), d.min_block, d.slots, &g)) return BQ_ERR_SIZE;
    bqx_tx* tx = new (std::nothrow) bqx_tx();
    if (!tx) return BQ_ERR_CUDA;
    tx->cb = cb;
    tx->g = g;
    tx->mode = mode;
    tx->rx_device = d.device;
    tx->remote_process = (d.pid != int32_t(getpid()));
    cudaError_t e = cudaGetDevice(&tx->device);
    if (e != cudaSuccess) { delete tx; return cuda_fail(e); }
    if (!tx->remote_process) {
        if (tx->device != d.device) {
            int can = 0;
            e = cudaDeviceCanAccessPeer(&can, tx->device, d.device);
            if (e != cudaSuccess) { delete tx; return cuda_fail(e); }
            if (!can) {
                delete tx;
                char text[128];
                std::snprintf(text, sizeof(text), "bqx_tx_open: device %d cannot reach device %d's memory (no peer access)", tx->device, d.device);
                return fail_text(text);
            }
            e = cudaDeviceEnablePeerAccess(d.device, 0);
            if (e == cudaErrorPeerAccessAlreadyEnabled) { (void)cudaGetLastError(); e = cudaSuccess; }
            if (e != cudaSuccess) { delete tx; return cuda_fail(e); }
        }
        tx->mailbox = reinterpret_cast<char*>(uintptr_t(d.mailbox));
        for (int s = 0; s < g.slots; ++s) {
            tx->filled[s] = reinterpret_cast<cudaEvent_t>(uintptr_t(d.filled[s]));
            tx->drained[s] = reinterpret_cast<cudaEvent_t>(uintptr_t(d.drained[s]));
        }
    } else {
        if (!d.have_ipc) { delete tx; return fail_text("bqx_tx_open: the mailbox belongs to another process and carries no IPC handles"); }
        void* p = nullptr;
        e = cudaIpcOpenMemHandle(&p, d.mem, cudaIpcMemLazyEnablePeerAccess);
        for (int s = 0; s < g.slots && e == cudaSuccess; ++s) {
            e = cudaIpcOpenEventHandle(&tx->filled[s], d.filled_ipc[s]);
            if (e == cudaSuccess) e = cudaIpcOpenEventHandle(&tx->drained[s], d.drained_ipc[s]);
        }
        if (e != cudaSuccess) {
            if (p) cudaIpcCloseMemHandle(p);
            delete tx;
            return cuda_fail(e);
        }
        tx->mailbox = static_cast<char*>(p);
    }
    if (mode == BQX_COPY) {
        e = cudaMalloc(reinterpret_cast<void**>(&tx->staging), g.slot_bytes * size_t(g.slots));
        if (e != cudaSuccess) { bqx_tx_close(tx); return cuda_fail(e); }
    }
    *out = tx;
    return BQ_OK;
}

int bqx_tx_close(bqx_tx* tx) {
    if (!tx) return BQ_OK;
    cudaError_t e = cudaSuccess;
    if (tx->staging) e = cudaFree(tx->staging);
    if (tx->remote_process) {
        for (int s = 0; s < tx->g.slots; ++s) {
            if (tx->filled[s]) cudaEventDestroy(tx->filled[s]);
            if (tx->drained[s]) cudaEventDestroy(tx->drained[s]);
        }
        if (tx->mailbox) cudaIpcCloseMemHandle(tx->mailbox);
    }
    delete tx;
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bqx_tx_send_piece(bqx_tx* tx, const void* x_piece, bq_dtype xdt, size_t count, int block, int slot, void* cuda_stream) {
    if (!tx) return BQ_ERR_NULL;
    if (!known_dtype(xdt)) return BQ_ERR_DTYPE;
    if (block < tx->g.min_block || size_t(block) > tx->g.chunk) return BQ_ERR_BLOCK;
    if (count > tx->g.chunk || slot < 0 || slot >= tx->g.slots) return BQ_ERR_SIZE;
    if (count == 0) return BQ_OK;
    if (!x_piece) return BQ_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* dst = tx->mailbox + tx->g.slot_bytes * size_t(slot);
    if (tx->used[slot]) BQ_TRY(cudaStreamWaitEvent(stream, tx->drained[slot], 0));
    if (tx->mode == BQX_STORE) {
        const int rc = bq_quantize(x_piece, xdt, count, block, tx->cb, reinterpret_cast<uint8_t*>(dst),
                                   reinterpret_cast<float*>(dst + tx->g.codes_bytes), stream);
        if (rc != BQ_OK) return rc;
    } else {
        char* st = tx->staging + tx->g.slot_bytes * size_t(slot);
        const int rc = bq_quantize(x_piece, xdt, count, block, tx->cb, reinterpret_cast<uint8_t*>(st),
                                   reinterpret_cast<float*>(st + tx->g.codes_bytes), stream);
        if (rc != BQ_OK) return rc;
        const size_t nb = (count + size_t(block) - 1) / size_t(block);
        // cudaMemcpyDefault: the unified address space tells the runtime which devices the two ends are on
        BQ_TRY(cudaMemcpyAsync(dst, st, count, cudaMemcpyDefault, stream));
        BQ_TRY(cudaMemcpyAsync(dst + tx->g.codes_bytes, st + tx->g.codes_bytes, nb * 4, cudaMemcpyDefault, stream));
    }
    BQ_TRY(cudaEventRecord(tx->filled[slot], stream));
    tx->used[slot] = true;
    return BQ_OK;
}

int bqx_rx_recv_piece(bqx_rx* rx, size_t count, int block, int slot, void* y_piece, bq_dtype ydt, void* cuda_stream) {
    if (!rx) return BQ_ERR_NULL;
    if (!known_dtype(ydt)) return BQ_ERR_DTYPE;
    if (block < rx->g.min_block || size_t(block) > rx->g.chunk) return BQ_ERR_BLOCK;
    if (count > rx->g.chunk || slot < 0 || slot >= rx->g.slots) return BQ_ERR_SIZE;
    if (count == 0) return BQ_OK;
    if (!y_piece) return BQ_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const char* src = rx->mailbox + rx->g.slot_bytes * size_t(slot);
    BQ_TRY(cudaStreamWaitEvent(stream, rx->filled[slot], 0));
    const int rc = bq_dequantize(reinterpret_cast<const uint8_t*>(src), reinterpret_cast<const float*>(src + rx->g.codes_bytes), count, block,
                                 rx->cb, y_piece, ydt, stream);
    if (rc != BQ_OK) return rc;
    BQ_TRY(cudaEventRecord(rx->drained[slot], stream));
    return BQ_OK;
}

int bqx_transfer(bqx_tx* tx, bqx_rx* rx, const void* x, bq_dtype xdt, size_t n, int block, void* y_out, bq_dtype ydt, void* send_stream,
                 void* recv_stream) {
    if (!tx || !rx) return BQ_ERR_NULL;
    if (!known_dtype(xdt) || !known_dtype(ydt)) return BQ_ERR_DTYPE;
    if (tx->remote_process || tx->g.chunk != rx->g.chunk || tx->g.slots != rx->g.slots || tx->g.min_block != rx->g.min_block) return BQ_ERR_SIZE;
    if (block < rx->g.min_block || size_t(block) > rx->g.chunk) return BQ_ERR_BLOCK;
    if (n >= (size_t(1) << 40)) return BQ_ERR_SIZE;
    if (n == 0) return BQ_OK;
    if (!x || !y_out) return BQ_ERR_NULL;
    const int xs = xdt == BQ_F32 ? 4 : 2, ys = ydt == BQ_F32 ? 4 : 2;
    int here = -1;
    BQ_TRY(cudaGetDevice(&here));
    size_t pieces = 0;
    int rc = bqx_plan(n, block, rx->g.chunk, rx->g.slots, 0, &pieces, nullptr, nullptr, nullptr);
    for (size_t p = 0; p < pieces && rc == BQ_OK; ++p) {
        int slot = 0;
        size_t first = 0, count = 0;
        rc = bqx_plan(n, block, rx->g.chunk, rx->g.slots, p, nullptr, &slot, &first, &count);
        if (rc != BQ_OK) break;
        // the codebook handles belong to their devices, and so do the streams
        if (cudaSetDevice(tx->device) != cudaSuccess) { rc = cuda_fail(cudaGetLastError()); break; }
        rc = bqx_tx_send_piece(tx, static_cast<const char*>(x) + first * xs, xdt, count, block, slot, send_stream);
        if (rc != BQ_OK) break;
        if (cudaSetDevice(rx->device) != cudaSuccess) { rc = cuda_fail(cudaGetLastError()); break; }
        rc = bqx_rx_recv_piece(rx, count, block, slot, static_cast<char*>(y_out) + first * ys, ydt, recv_stream);
    }
    cudaSetDevice(here);
    return rc;
}

}  // extern "C"
