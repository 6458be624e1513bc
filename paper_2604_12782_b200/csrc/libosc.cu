// Single translation unit of the library: the kernels share one device-side status word, so they
// are compiled together (no relocatable device code needed).
#include "quant_kernels.cu"
#include "norm_kernels.cu"
#include "gemm_kernels.cu"
#include "gemm2_kernels.cu"
#include "gemm3_kernels.cu"
#include "profile_kernels.cu"
#include "api.cu"
#include "static_scratch.cu"
