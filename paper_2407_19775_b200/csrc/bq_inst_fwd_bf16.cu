// Tuned forward kernels for bf16 tensors.
#define BQ_INST_DT bqk::kBF16
#define BQ_INST_NAME launch_fwd_fast_bf16
#include "bq_fwd_inst.cuh"
