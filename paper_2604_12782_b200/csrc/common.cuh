// Declarations shared by the translation units of the library (host side + kernel launchers).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "ptx.cuh"

namespace osc {

// Launch with programmatic stream serialization allowed: the kernel may begin (up to its
// grid_dependency_wait) while the previous kernel on the stream is finishing.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Function attributes (the shared-memory opt-in) and occupancy answers belong to a device, not to the process:
// every kernel instantiation keeps one of these and sets itself up once on each device it is launched on.
constexpr int kMaxDevicesPerProcess = 64;
struct PerDevice {   // threads may race to fill a slot: both then store the same values, and a reader that sees
                     // `done` also sees `value` (sequentially consistent atomics)
    std::atomic<bool> done[kMaxDevicesPerProcess] = {};
    std::atomic<int> value[kMaxDevicesPerProcess] = {};
};
// index of the current device in a PerDevice, or -1 (no caching) if it cannot be had or is out of range
static inline int per_device_slot() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevicesPerProcess) return -1;
    return dev;
}
template <typename Kernel>
static cudaError_t opt_in_shared_memory(PerDevice& pd, Kernel kernel, int bytes) {
    const int slot = per_device_slot();
    if (slot >= 0 && pd.done[slot]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && slot >= 0) pd.done[slot] = true;
    return e;
}

// quant_kernels.cu
cudaError_t launch_quant_extract(const CUtensorMap& tm_x, int M, int K, const uint32_t* mask,
                                 const int32_t* prefix, const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko, int Kop,
                                 const int32_t* sched, int max_tiles, int num_sms, cudaStream_t st);
cudaError_t launch_quant_extract_nvfp4(const CUtensorMap& tm_x, int M, int K, const uint32_t* mask,
                                       const int32_t* prefix, const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko,
                                       int Kop, int num_sms, int tensor_e, cudaStream_t st,
                                       const int32_t* sched = nullptr, int max_tiles = 0);
cudaError_t launch_fp8_quant(const void* X, int64_t ldx, int M, int K, void* x8, void* sx, cudaStream_t st);
cudaError_t launch_mxfp8_quant(const void* X, int64_t ldx, int M, int K, void* x8, void* sf, const int32_t* sched,
                               int max_tiles, cudaStream_t st);
cudaError_t launch_dyn_quant_extract(const void* X, int64_t ldx, int M, int K, void* xq, void* sf, void* xo, void* idx,
                                     void* val, cudaStream_t st);
cudaError_t launch_build_sched(const int32_t* off, int E, int32_t* sched128, int max_tiles128, int32_t* sched256,
                               int max_tiles256, cudaStream_t st);

cudaError_t launch_prepare_fence(cudaStream_t st);   // last launch of every weight preparation

// sf_channels: channels per scale block (128 for MXFP4, 64 for NVFP4)
cudaError_t launch_gather_quantized(const int32_t* row_token, int T, int K, int Kop, const void* xq_u, const void* sf_u,
                                    const void* xo_u, void* xq, void* sf, void* xo, const int32_t* sched, int max_tiles,
                                    cudaStream_t st, int sf_channels = 128);

// norm_kernels.cu
cudaError_t launch_rmsnorm_quant(bool quant, const void* H, int64_t ldh, int M, int K, const void* gamma, float eps,
                                 void* Xn, int64_t ldx, const int32_t* idx_o, void* xq, void* sf,
                                 void* xo, int Ko, int Kop, cudaStream_t st, const void* R = nullptr, int64_t ldr = 0,
                                 void* Hout = nullptr, int64_t ldo = 0);

cudaError_t launch_rmsnorm_quant_nvfp4(const void* H, int64_t ldh, int M, int K, const void* gamma, float eps,
                                       const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko, int Kop, int tensor_e,
                                       cudaStream_t st);

cudaError_t launch_swiglu_fp8(bool quant, const void* GU, int64_t ldg, int M, int I, void* Hout, int64_t ldh, void* x8,
                              void* sx, cudaStream_t st);

// profile_kernels.cu
cudaError_t launch_profile(const void* X, int64_t ldx, int S, int K, double alpha, double* sum, int32_t* counts,
                           int8_t* lut, int32_t* n_hit, int32_t* n_total, uint32_t* threshold_bits, int num_sms,
                           cudaStream_t st);

// gemm_kernels.cu
struct GemmArgs {
    CUtensorMap tm_a;    // Path A activations: packed FP4 bytes [rows, K/2]  (FP8 mode: [rows, K])
    CUtensorMap tm_b;    // Path A weights    : [E*N, K/2]                    (FP8 mode: [E*N, K])
    CUtensorMap tm_ao;   // Path B activations: bf16 [rows, K_o_pad]
    CUtensorMap tm_bo;   // Path B weights    : bf16 [E*N, K_o_pad]
    CUtensorMap tm_sfa;  // activation scale blocks as uint32 [blocks, 128] (CTA-pair kernel only)
    CUtensorMap tm_sfw;  // weight scale blocks, same form
    CUtensorMap tm_y;    // output bf16 [rows, ldy], 32 x 64 store tiles (CTA-pair kernel only)
    CUtensorMap tm_y16;  // the same with 16 x 64 store tiles (240-wide tiles of the CTA-pair kernel)
    const uint8_t* sfa;  // activation scales, block layout
    const uint8_t* sfw;  // weight scales, block layout, per expert
    const float* sx;     // FP8 mode: per-row activation scale
    const float* sw;     // FP8 mode: per-output-row weight scale [E*N]
    float out_scale;     // NVFP4 mode: product of the two power-of-two tensor scales, applied before the bf16 rounding
    uint16_t* Y;         // bf16 [rows, ldy]
    int64_t ldy;
    int M;               // rows (dense) / total rows (grouped)
    int N, K, Kop;
    const int32_t* sched;  // grouped tile schedule (128-row tiles) or nullptr
    int max_tiles;
    const int32_t* sched2; // grouped tile schedule of the CTA-pair kernel (256-row tiles) or nullptr
    int max_tiles2;
    int num_sms;
    int band;            // CTA-pair kernel: 256-row tiles per scheduling band (set by its launcher)
};
cudaError_t launch_gemm_dual(const GemmArgs& a, int bn, cudaStream_t st);
cudaError_t launch_gemm_fp8(const GemmArgs& a, int bn, cudaStream_t st);
cudaError_t launch_gemm_mxf8(const GemmArgs& a, int bn, cudaStream_t st);
cudaError_t launch_gemm_nvf4(const GemmArgs& a, int bn, cudaStream_t st);
int gemm_block_n(int row_tiles, int N, int num_sms, long* cost_ns = nullptr, int widest = 256);

// gemm2_kernels.cu (CTA pairs: 256-row tiles, dense or grouped)
cudaError_t launch_gemm_dual_pair(const GemmArgs& a, int bn, cudaStream_t st);
cudaError_t launch_gemm_fp8_pair(const GemmArgs& a, int bn, cudaStream_t st);
cudaError_t launch_gemm_dual_pair_swiglu(const GemmArgs& a, cudaStream_t st);
cudaError_t launch_gemm_mxf8_pair(const GemmArgs& a, int bn, cudaStream_t st);
cudaError_t launch_gemm_nvf4_pair(const GemmArgs& a, int bn, cudaStream_t st);
int gemm_pair_block_n(bool fp8, bool allow_240, long row_tiles, int N, int stages, int num_sms, long* cost_ns = nullptr);

// gemm3_kernels.cu (few rows: operands swapped, K split over a cluster)
// activations of the few-row kernel's in-kernel quantizer (Algorithm 2 on the CTA's own K slice)
struct DecodeX {
    const uint16_t* X;     // bf16 [M, ldx]
    int64_t ldx;
    const uint32_t* mask;  // flagged channels per 32-channel group
    const int32_t* idx_o;  // channel of every column of the buffer B
    int Ko;
};
cudaError_t launch_gemm_dual_decode(const GemmArgs& a, int S, cudaStream_t st);
cudaError_t launch_gemm_dual_decode_quant(const GemmArgs& a, const DecodeX& xa, int S, cudaStream_t st);
cudaError_t launch_gemm_fp8_decode(const GemmArgs& a, int S, cudaStream_t st);
cudaError_t launch_gemm_mxf8_decode(const GemmArgs& a, int S, cudaStream_t st);
cudaError_t launch_gemm_nvf4_decode(const GemmArgs& a, int S, cudaStream_t st);
int gemm_decode_split(int N, int nkb, int num_sms);
cudaError_t launch_retile_sf(const uint8_t* src, uint8_t* dst, int N, int K, int bn, cudaStream_t st, bool gate_up = false,
                             int sf_channels = 128);

}  // namespace osc
