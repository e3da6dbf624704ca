// bq_host.cu -- the host-buffer calls of include/bq.h: a chunked three-stream pipeline between
// host buffers around the device-pointer calls.  This file moves bytes and orders streams; the
// method's arithmetic is all in the kernels behind bq_quantize / bq_dequantize / bq_roundtrip.
//
// Per piece p (slot s = p mod slots):
//     up stream:    wait free[s] (the slot's previous download)   copy in   record in[s]
//     run stream:   wait in[s]                                    kernel    record ran[s]
//     down stream:  wait ran[s]                                   copy out  record free[s]
// Calls on one pipe take effect in order without waiting for each other more than they must.  The
// three streams are each in order, the slots are guarded by their events, and a call ends by
// recording `done` on the down stream (which has by then waited for everything else of the
// call).  What the streams' own order does not give is a later call READING host memory that an
// earlier, still unfinished call WRITES (the receiver expanding what the sender just produced):
// the pipe remembers the host ranges its unfinished calls write, and a call whose inputs overlap
// one of them first makes its uploads wait for `done`.  Otherwise the uploads of a call run under
// the downloads of the call before it.
#include "../../include/bq.h"
#include "bq_error.h"

#include <cuda_runtime.h>

#include <new>

struct bq_host_pipe {
    const bq_codebook* cb;
    int device;
    size_t chunk;            // elements per piece at most
    int min_block;
    int elem_bytes;          // bytes per element of the staging buffers
    int slots;
    char* blob;              // one device allocation: per slot x | y | codes | absmax
    char* x[8];
    char* y[8];
    uint8_t* codes[8];
    float* absmax[8];
    cudaStream_t up, run, down;
    cudaEvent_t in[8], ran[8], free_[8], done;
    bool used[8];            // the slot has a download in flight or behind it (free_[s] has been recorded)
    bool any;                // `done` has been recorded
    // host ranges written by calls enqueued since the last wait on `done`
    const char* out_lo[24];
    const char* out_hi[24];
    int n_out;
};

namespace {

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

int bytes_of(int dt) { return dt == BQ_F32 ? 4 : 2; }
bool known_dtype(int dt) { return dt == BQ_F32 || dt == BQ_F16 || dt == BQ_BF16; }
size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool on_pipe_device(const bq_host_pipe* p) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == p->device;
}

enum Op { kQuantize, kDequantize, kRoundtrip };

struct Call {
    Op op;
    const char* x;           // host, elements of xdt
    char* y;                 // host, elements of ydt
    const uint8_t* codes_in; // host
    uint8_t* codes_out;      // host
    const float* absmax_in;  // host
    float* absmax_out;       // host
    int xdt, ydt;
};

#define BQ_TRY(expr)                                   \
    do {                                               \
        const cudaError_t e_ = (expr);                 \
        if (e_ != cudaSuccess) return cuda_fail(e_);   \
    } while (0)

bool overlaps(const bq_host_pipe* p, const void* lo, size_t bytes) {
    const char* a = static_cast<const char*>(lo);
    for (int i = 0; i < p->n_out; ++i)
        if (a < p->out_hi[i] && p->out_lo[i] < a + bytes) return true;
    return false;
}

void remember_output(bq_host_pipe* p, void* lo, size_t bytes) {
    p->out_lo[p->n_out] = static_cast<const char*>(lo);
    p->out_hi[p->n_out] = static_cast<const char*>(lo) + bytes;
    ++p->n_out;
}

int run_call(bq_host_pipe* p, const Call& c, size_t n, int block) {
    const size_t B = size_t(block);
    const size_t piece = (p->chunk / B) * B;          // whole blocks per piece
    const int xs = bytes_of(c.xdt), ys = bytes_of(c.ydt);
    const size_t nblocks = (n + B - 1) / B;
    // does this call read what an unfinished call writes?  (or is the list of remembered ranges full?)
    bool must_wait = p->n_out + 2 > 24;
    if (c.op == kDequantize) must_wait = must_wait || overlaps(p, c.codes_in, n) || overlaps(p, c.absmax_in, nblocks * 4);
    else must_wait = must_wait || overlaps(p, c.x, n * size_t(xs));
    if (p->any && must_wait) {
        BQ_TRY(cudaStreamWaitEvent(p->up, p->done, 0));          // everything enqueued so far has finished before the first upload
        p->n_out = 0;
    }
    if (c.op == kQuantize) {
        remember_output(p, c.codes_out, n);
        remember_output(p, c.absmax_out, nblocks * 4);
    } else {
        remember_output(p, c.y, n * size_t(ys));
    }
    size_t i = 0;
    for (size_t lo = 0; lo < n; lo += piece, ++i) {
        const int s = int(i % size_t(p->slots));
        const size_t cnt = (n - lo < piece) ? n - lo : piece;
        const size_t b0 = lo / B, nb = (cnt + B - 1) / B;
        if (p->used[s]) BQ_TRY(cudaStreamWaitEvent(p->up, p->free_[s], 0));
        if (c.op == kDequantize) {
            BQ_TRY(cudaMemcpyAsync(p->codes[s], c.codes_in + lo, cnt, cudaMemcpyHostToDevice, p->up));
            BQ_TRY(cudaMemcpyAsync(p->absmax[s], c.absmax_in + b0, nb * 4, cudaMemcpyHostToDevice, p->up));
        } else {
            BQ_TRY(cudaMemcpyAsync(p->x[s], c.x + lo * xs, cnt * xs, cudaMemcpyHostToDevice, p->up));
        }
        BQ_TRY(cudaEventRecord(p->in[s], p->up));
        BQ_TRY(cudaStreamWaitEvent(p->run, p->in[s], 0));
        int rc;
        if (c.op == kQuantize) rc = bq_quantize(p->x[s], bq_dtype(c.xdt), cnt, block, p->cb, p->codes[s], p->absmax[s], p->run);
        else if (c.op == kDequantize) rc = bq_dequantize(p->codes[s], p->absmax[s], cnt, block, p->cb, p->y[s], bq_dtype(c.ydt), p->run);
        else rc = bq_roundtrip(p->x[s], bq_dtype(c.xdt), cnt, block, p->cb, p->y[s], bq_dtype(c.ydt), nullptr, nullptr, p->run);
        if (rc != BQ_OK) return rc;
        BQ_TRY(cudaEventRecord(p->ran[s], p->run));
        BQ_TRY(cudaStreamWaitEvent(p->down, p->ran[s], 0));
        if (c.op == kQuantize) {
            BQ_TRY(cudaMemcpyAsync(c.codes_out + lo, p->codes[s], cnt, cudaMemcpyDeviceToHost, p->down));
            BQ_TRY(cudaMemcpyAsync(c.absmax_out + b0, p->absmax[s], nb * 4, cudaMemcpyDeviceToHost, p->down));
        } else {
            BQ_TRY(cudaMemcpyAsync(c.y + lo * ys, p->y[s], cnt * ys, cudaMemcpyDeviceToHost, p->down));
        }
        BQ_TRY(cudaEventRecord(p->free_[s], p->down));
        p->used[s] = true;
    }
    // the down stream has waited for every kernel of the call, and each kernel for its upload
    BQ_TRY(cudaEventRecord(p->done, p->down));
    p->any = true;
    return BQ_OK;
}

int check_call(const bq_host_pipe* p, int dt, size_t n, int block) {
    if (!p) return BQ_ERR_NULL;
    if (!known_dtype(dt)) return BQ_ERR_DTYPE;
    if (bytes_of(dt) > p->elem_bytes) return BQ_ERR_DTYPE;
    if (block < 1 || block < p->min_block || size_t(block) > p->chunk) return BQ_ERR_BLOCK;
    if (n >= (size_t(1) << 40)) return BQ_ERR_SIZE;
    return BQ_OK;
}

void release(bq_host_pipe* p) {
    for (int s = 0; s < 8; ++s) {
        if (p->in[s]) cudaEventDestroy(p->in[s]);
        if (p->ran[s]) cudaEventDestroy(p->ran[s]);
        if (p->free_[s]) cudaEventDestroy(p->free_[s]);
    }
    if (p->done) cudaEventDestroy(p->done);
    if (p->up) cudaStreamDestroy(p->up);
    if (p->run) cudaStreamDestroy(p->run);
    if (p->down) cudaStreamDestroy(p->down);
    if (p->blob) cudaFree(p->blob);
    delete p;
}

}  // namespace

extern "C" {

int bq_host_pipe_create(const bq_codebook* cb, size_t chunk_elems, int min_block, bq_dtype widest, int slots, bq_host_pipe** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (!known_dtype(widest)) return BQ_ERR_DTYPE;
    if (min_block < 1 || size_t(min_block) > chunk_elems) return BQ_ERR_BLOCK;
    if (chunk_elems == 0 || chunk_elems >= (size_t(1) << 34) || slots < 2 || slots > 8) return BQ_ERR_SIZE;
    bq_host_pipe* p = new (std::nothrow) bq_host_pipe();
    if (!p) return BQ_ERR_CUDA;
    p->cb = cb;
    p->chunk = chunk_elems;
    p->min_block = min_block;
    p->elem_bytes = bytes_of(widest);
    p->slots = slots;
    cudaError_t e = cudaGetDevice(&p->device);
    const size_t xb = round_up(chunk_elems * size_t(p->elem_bytes), 256), cbytes = round_up(chunk_elems, 256);
    const size_t ab = round_up((chunk_elems / size_t(min_block) + 1) * 4, 256);
    const size_t per_slot = 2 * xb + cbytes + ab;
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&p->blob), per_slot * size_t(slots));
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->up, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->run, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->down, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->done, cudaEventDisableTiming);
    for (int s = 0; s < slots && e == cudaSuccess; ++s) {
        char* base = p->blob + per_slot * size_t(s);
        p->x[s] = base;
        p->y[s] = base + xb;
        p->codes[s] = reinterpret_cast<uint8_t*>(base + 2 * xb);
        p->absmax[s] = reinterpret_cast<float*>(base + 2 * xb + cbytes);
        e = cudaEventCreateWithFlags(&p->in[s], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ran[s], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->free_[s], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        release(p);
        return cuda_fail(e);
    }
    *out = p;
    return BQ_OK;
}

int bq_host_pipe_destroy(bq_host_pipe* p) {
    if (!p) return BQ_OK;
    cudaError_t e = cudaSuccess;
    if (p->any) e = cudaEventSynchronize(p->done);
    release(p);
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bq_quantize_host(bq_host_pipe* p, const void* x_host, bq_dtype xdt, size_t n, int block, uint8_t* codes_host, float* absmax_host) {
    const int rc = check_call(p, xdt, n, block);
    if (rc != BQ_OK) return rc;
    if (n == 0) return BQ_OK;
    if (!x_host || !codes_host || !absmax_host) return BQ_ERR_NULL;
    if (!on_pipe_device(p)) return BQ_ERR_CODEBOOK;
    Call c = {kQuantize, static_cast<const char*>(x_host), nullptr, nullptr, codes_host, nullptr, absmax_host, xdt, xdt};
    return run_call(p, c, n, block);
}

int bq_dequantize_host(bq_host_pipe* p, const uint8_t* codes_host, const float* absmax_host, size_t n, int block, void* y_host, bq_dtype ydt) {
    const int rc = check_call(p, ydt, n, block);
    if (rc != BQ_OK) return rc;
    if (n == 0) return BQ_OK;
    if (!codes_host || !absmax_host || !y_host) return BQ_ERR_NULL;
    if (!on_pipe_device(p)) return BQ_ERR_CODEBOOK;
    Call c = {kDequantize, nullptr, static_cast<char*>(y_host), codes_host, nullptr, absmax_host, nullptr, ydt, ydt};
    return run_call(p, c, n, block);
}

int bq_roundtrip_host(bq_host_pipe* p, const void* x_host, bq_dtype xdt, size_t n, int block, void* y_host, bq_dtype ydt) {
    int rc = check_call(p, xdt, n, block);
    if (rc == BQ_OK) rc = check_call(p, ydt, n, block);
    if (rc != BQ_OK) return rc;
    if (n == 0) return BQ_OK;
    if (!x_host || !y_host) return BQ_ERR_NULL;
    if (!on_pipe_device(p)) return BQ_ERR_CODEBOOK;
    Call c = {kRoundtrip, static_cast<const char*>(x_host), static_cast<char*>(y_host), nullptr, nullptr, nullptr, nullptr, xdt, ydt};
    return run_call(p, c, n, block);
}

int bq_host_pipe_wait(bq_host_pipe* p) {
    if (!p) return BQ_ERR_NULL;
    if (!p->any) return BQ_OK;
    const cudaError_t e = cudaEventSynchronize(p->done);
    p->n_out = 0;                                         // nothing is unfinished any more
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bq_host_pipe_wait_on_stream(bq_host_pipe* p, void* cuda_stream) {
    if (!p) return BQ_ERR_NULL;
    if (!p->any) return BQ_OK;
    const cudaError_t e = cudaStreamWaitEvent(static_cast<cudaStream_t>(cuda_stream), p->done, 0);
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

}  // extern "C"
