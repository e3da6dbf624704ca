// Tuned forward kernels for f16 tensors.
#define BQ_INST_DT bqk::kF16
#define BQ_INST_NAME launch_fwd_fast_f16
#include "bq_fwd_inst.cuh"
