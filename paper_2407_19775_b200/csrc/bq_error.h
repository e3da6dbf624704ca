// bq_error.h -- the per-thread text behind bq_last_cuda_error (internal to libbq).
#pragma once

namespace bql {
void set_last_cuda_error(const char* text);
}
