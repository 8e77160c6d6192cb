// Single translation unit of libpquant.so: the kernels share one device status
// word and are compiled together (no relocatable device code needed).
#include "pq_elementwise.cu"
#include "pq_gemm_kernels.cu"
#include "pq_decode.cu"
#include "pq_decode_stream.cu"
#include "pq_api.cu"
