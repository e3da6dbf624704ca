// bq_debug.h -- host-side assertions of a debug build of the library (compile the API units with
// -DBQ_DEBUG; `python -m paper_2407_19775_b200.build --debug` links them into libbq_debug.so).
//
// A debug build checks, before anything is enqueued, what a release build takes on trust: that the
// caller's buffers do not overlap in a way the kernels do not allow (an output over another output,
// an output over an input other than the documented in-place roundtrip), and that the split of the
// tensor between the tuned kernel and the general one covers every element once (the tuned part a
// whole number of blocks, the rest starting on a block border, nothing past n).  A failed assertion
// returns BQ_ERR_ASSERT with the failed condition as the last error text; nothing is launched.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include "bq.h"
#include "bq_error.h"

namespace bqd {

#ifdef BQ_DEBUG
constexpr bool kOn = true;
#else
constexpr bool kOn = false;
#endif

// [a, a + an) and [b, b + bn) share no byte (empty ranges never do)
inline bool disjoint(const void* a, size_t an, const void* b, size_t bn) {
    if (!a || !b || an == 0 || bn == 0) return true;
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 + an <= b0 || b0 + bn <= a0;
}

}  // namespace bqd

#define BQ_ASSERT(cond)                                                      \
    do {                                                                     \
        if (bqd::kOn && !(cond)) {                                           \
            bql::set_last_cuda_error("debug assertion failed: " #cond);      \
            return BQ_ERR_ASSERT;                                            \
        }                                                                    \
    } while (0)
