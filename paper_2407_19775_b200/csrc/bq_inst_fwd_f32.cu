// Tuned forward kernels for f32 tensors.
#define BQ_INST_DT bqk::kF32
#define BQ_INST_NAME launch_fwd_fast_f32
#include "bq_fwd_inst.cuh"
