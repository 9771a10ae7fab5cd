#include "lrq_internal.cuh"
lrq_status lrq_launch_qgemm_tc(const lrq_layer*, const uint8_t*, const float*, const int32_t*, int, void*, lrq_dtype,
                               long, cudaStream_t) { return LRQ_ERR_UNSUPPORTED; }
