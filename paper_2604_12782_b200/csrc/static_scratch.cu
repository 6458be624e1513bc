// osc_linear_static: the OSC linear for callers that cannot provide a workspace.
//
// osc_linear needs scratch memory between its two kernels (packed codes, scale blocks and the
// gathered channels).  Some callers have no way to get device memory for it: a plug-in that its
// host framework hands nothing but input and output pointers, or code on a path where an
// allocation (and the device-wide synchronisation cudaMalloc implies) is not acceptable.  For them
// the scratch lives in the fixed array below, which every GPU that loads this library holds until
// the process exits.
#include "../../include/osc.h"
#include "common.cuh"

// File-scope device array.  In host code this name is only a stand-in for the symbol; the device
// address has to be asked for with cudaGetSymbolAddress (per device) before it is given to a kernel.
static __device__ __align__(256) unsigned char g_osc_static_scratch[OSC_STATIC_SCRATCH_BYTES];

namespace osc {

// Device address of the scratch array on the current device.  Asked for on every call (a host-side table lookup in
// the runtime): nothing is cached here, so host threads need no coordination and a context that was torn down and
// created again is served with its own copy of the array.
static osc_status static_scratch_address(void** out) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_osc_static_scratch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
    if (!p) return fail(OSC_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
    *out = p;
    return OSC_OK;
}

}  // namespace osc

extern "C" osc_status osc_linear_static(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y,
                                        int64_t ldy, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights are not supported by osc_linear_static");
    if (M == 0) return OSC_OK;
    osc_act_sizes_t sz;
    osc_act_sizes(w, M, &sz);
    if (sz.workspace_bytes > (size_t)OSC_STATIC_SCRATCH_BYTES)
        return fail(OSC_ERR_WORKSPACE,
                    "osc_linear_static: M = %d with K = %d, K_o_pad = %d needs %zu bytes of scratch, the built-in array "
                    "holds %d; use osc_linear with a caller workspace",
                    M, w->K, w->Kop, sz.workspace_bytes, OSC_STATIC_SCRATCH_BYTES);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    void* base = nullptr;
    if (osc_status s = static_scratch_address(&base)) return s;
    uint8_t* ws = static_cast<uint8_t*>(base);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Nothing in the scratch has to start at zero: the quantizer writes every byte the GEMM reads
    // (codes and gathered channels of all M rows, pad columns, whole scale blocks incl. rows past M).
    if (osc_status s = quantize_impl(w, X, M, ldx, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, nullptr, 0, st))
        return s;
    return gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M, Y, ldy, nullptr, 0, nullptr, 0, st);
}
