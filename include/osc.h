/*
 * osc.h - C ABI of the B200 (sm_100a) OSC dual-path quantized linear layer.
 *
 * The calls follow the paper's statement of the problem:
 *   offline  : suppression table + weight split            (Section 3.1; Section 3.3 "offline weight quantization")
 *   online   : OSC-enhanced quantization                   (Algorithm 2)
 *              dual-path GEMM  Y = (Q_X (x) Q_W).S + B.W_L (Eq. 5)
 *   fallback : FP8 W8A8 linear for the down-projection     (Section 3.4)
 *   grouped  : the same linears per MoE expert             (Section 4.1, Qwen3-30B-A3B: 128 experts, 8 active)
 *
 * Conventions
 *   - Plain C, no exceptions cross the boundary.  Every call returns an osc_status
 *     (0 = success, negative = error); osc_last_error() gives a thread-local detail string.
 *   - "dev" pointers are device (HBM) addresses, "host" pointers are host addresses.
 *     The caller owns every device buffer.  The library allocates no device memory and keeps
 *     only small host handles (shapes, borrowed device pointers, TMA descriptors) created by
 *     *_prepare_* and released by *_destroy.
 *   - stream is a cudaStream_t passed as void*.  All work is enqueued on it; no call
 *     synchronizes except osc_sync_check.  A failed validation launches nothing.
 *     Kernels are launched with programmatic stream serialization (a kernel's prologue may overlap its
 *     predecessor's tail, and the few-row GEMM streams weights ahead of its dependency wait); every
 *     *_prepare_* call ends with a plain launch, so a handle may be used on the same stream directly behind
 *     its preparation without a synchronisation.  On another stream, order the use behind the preparation
 *     with an event as for any other stream work.
 *   - Devices: a handle belongs to the device that was current when it was prepared (its buffers live there and
 *     it remembers that device's SM count); call with that device current and a stream of that device.  One
 *     process per GPU is the intended arrangement: the path has no exchange step, so several GPUs run
 *     independent replicas (or disjoint row ranges of M) with no collective.
 *     cudaDeviceReset (or any other loss of the device's context) invalidates every handle made on that device
 *     and the kernel attributes the library set there: destroy the handles first and use a fresh process, or do not reset.
 *   - Threads: calls on distinct handles (or on one handle with distinct activation buffers and workspaces)
 *     may be made from several host threads at once; the library keeps no mutable state of its own beyond
 *     once-only caches (driver entry point, per-device kernel attributes) that are safe to race on.  Two
 *     calls that share a workspace must be ordered by the caller (one stream, or events).
 *   - Tensors: X bf16 [M, K] row-major (K contiguous, leading dimension ldx elements);
 *     W bf16 [N, K] row-major (the nn.Linear layout, Y = X . W^T); Y bf16 [M, N] (ldy elements).
 *   - Shape preconditions: K % 128 == 0, N % 64 == 0, M >= 0 (M == 0 is a successful no-op),
 *     device pointers 16-byte aligned, leading dimensions multiples of 8 elements.
 *   - Group size G = 32 (MXFP4).  The suppression table is lut[K/32][lut_c] int8 on the host:
 *     local channel index 0..31 or -1 (no channel).  lut_c = 1 is the paper's one channel per
 *     group; larger lut_c protects up to lut_c channels per group.
 *
 * Data layouts written by the library (and accepted back by osc_gemm_dual)
 *   xq / wq  : packed E2M1 codes, [rows, K/2] bytes, element 2i in bits 3:0 and 2i+1 in bits 7:4.
 *   sfa / sfw: E8M0 scale bytes, one per (row, 32-group), in 512-byte blocks of 128 rows x 4 groups:
 *              offset(r, g) = ((r/128)*(K/128) + g/4)*512 + (r%32)*16 + ((r%128)/32)*4 + g%4.
 *              Bytes of rows >= the row count are written as 0.
 *   xo / wo  : the protected channels, bf16 [rows, K_o_pad], ascending channel order,
 *              K_o_pad = roundup(K_o, 64), pad columns +0.
 *   meta     : uint32 mask[K/32], int32 prefix[K/32], int32 idx_o[K_o] (device copy of the table).
 *   x8 / w8  : E4M3 bytes [rows, K]; sx / sw: fp32 per-row scales (amax/448).
 *
 * Beyond the paper's main path, each in its own section below: the quantizers fused into their producers
 * (RMSNorm + Algorithm 2, SwiGLU + per-token FP8), the grouped form with the MoE dispatch fused behind the
 * quantizer, the MXFP8 form of the fallback, the NVFP4 / G = 16 form of the OSC path, the dynamic-protection
 * control group of Section 4.2 (a measured baseline), offline profiling (Algorithm 1), and osc_linear_static
 * (a deployment aid).
 *
 * Kernel selection is internal and depends only on the shape.  Few rows (M <= 32; <= 64 for layers with more
 * 128-feature tiles than SMs or a long K loop; <= 256 for long K loops with few tiles) run on a
 * weight-streaming kernel with the operands swapped and K split over a thread-block cluster; grouped problems
 * with large experts and dense problems with many tiles on 256-row CTA-pair tiles; the rest (up to 128 rows,
 * small experts, and dense problems whose 128-row tiles fit in one wave and beat the pair kernel's estimate) on
 * 128-row tiles.  The NVFP4 form runs on the same three kernels (few-row kernel up to 64 rows).  Results of
 * different kernels for the same inputs agree within the accumulation-order rounding of fp32, not bit for
 * bit; one kernel is deterministic run to run.
 * Environment variables for experiments (read by the library, not part of the contract): OSC_DECODE (0 = never,
 * 2 = always up to 256 rows), OSC_DECODE_SPLIT, OSC_DECODE_FUSED_ROWS (0 = the quantizer always its own kernel), OSC_PAIR (0 = 128-row tiles only, 2 = pair tiles whenever
 * eligible), OSC_PAIR_BLOCK_N, OSC_BLOCK_N, OSC_BAND, OSC_PAIRS, OSC_MAP_CACHE (0 = encode every TMA descriptor anew), OSC_LOG.
 * Sizes: M, N, K and E are ints; every row offset is computed in 64 bits, so M * K (and M * N) may exceed
 * 2^31 elements.
 */
#ifndef OSC_H_
#define OSC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int osc_status;
enum {
    OSC_OK = 0,
    OSC_ERR_INVALID_ARG = -1, /* null pointer, negative size, bad handle */
    OSC_ERR_SHAPE = -2,       /* K % 128, N % 64, leading dimension too small */
    OSC_ERR_LUT = -3,         /* table entry outside -1..31 or duplicated inside a group */
    OSC_ERR_ALIGN = -4,       /* pointer not 16-byte aligned / leading dimension not a multiple of 8 */
    OSC_ERR_WORKSPACE = -5,   /* workspace smaller than osc_*_act_sizes reports */
    OSC_ERR_ARCH = -6,        /* current device is not compute capability 10.x */
    OSC_ERR_CUDA = -7,        /* a CUDA runtime / driver call failed (detail in osc_last_error) */
    OSC_ERR_TIMEOUT = -8      /* a device-side wait gave up (reported by osc_sync_check) */
};

const char* osc_status_string(osc_status s);
const char* osc_last_error(void);

/* Waits for `stream` and reports OSC_ERR_TIMEOUT if any kernel of this library gave up on a
 * bounded device-side wait since the last check (the flag is cleared), OSC_ERR_CUDA if the
 * stream is in error, else OSC_OK.  Test / debugging aid; never needed on the hot path. */
osc_status osc_sync_check(void* stream);

/* ------------------------------------------------------------------ OSC path */

typedef struct osc_weights osc_weights; /* opaque host handle */

typedef struct {
    int32_t K_o;      /* protected channels listed in the table */
    int32_t K_o_pad;  /* roundup(K_o, 64) */
    size_t wq_bytes;  /* E * N * K/2 */
    size_t sfw_bytes; /* E * ceil(N/128) * (K/128) * 512 */
    size_t wo_bytes;  /* E * N * K_o_pad * 2 (0 when the table is empty) */
    size_t meta_bytes;
} osc_weight_sizes_t;

typedef struct {
    size_t xq_bytes;        /* M * K/2 */
    size_t sfa_bytes;       /* 512-byte scale blocks: ceil(M/128) row blocks (grouped: M/128 + E) x K/128 */
    size_t xo_bytes;        /* M * K_o_pad * 2 */
    size_t sched_bytes;     /* grouped only: device-built tile schedule */
    size_t xq_offset;       /* where osc_linear[_grouped] places each buffer inside its workspace */
    size_t sfa_offset;
    size_t xo_offset;
    size_t sched_offset;
    size_t workspace_bytes; /* total workspace osc_linear[_grouped] needs (each part 256-byte aligned) */
} osc_act_sizes_t;

/* Sizes of the buffers osc_prepare_weights[_grouped] fills (Section 3.3: FP4 weights plus
 * the gathered high-precision rows).  E = number of experts (1 for a dense layer).
 * lut: host [K/32][lut_c]. */
osc_status osc_weight_sizes(int E, int N, int K, const int8_t* lut, int lut_c, osc_weight_sizes_t* out);

/* Offline weight split (Section 3.3, first bullet; table semantics of Section 3.1):
 * W_o = W[:, idx_o]; W_r = W with those columns zeroed; (wq, sfw) = MXFP4(W_r).
 * W: dev bf16 [N, ldw].  wq/sfw/wo/meta: dev, caller-allocated with the sizes above; the
 * handle borrows them and they must outlive it.  Work is enqueued on `stream`. */
osc_status osc_prepare_weights(const void* W, int N, int K, int64_t ldw, const int8_t* lut, int lut_c,
                               void* wq, void* sfw, void* wo, void* meta, void* stream, osc_weights** out);

/* Same for E experts stacked as W[E][N][K] (dense, ldw = K); one table shared by all experts
 * of the layer; wq/sfw/wo are stacked per expert in the same order. */
osc_status osc_prepare_weights_grouped(const void* W, int E, int N, int K, const int8_t* lut, int lut_c,
                                       void* wq, void* sfw, void* wo, void* meta, void* stream,
                                       osc_weights** out);

osc_status osc_weights_destroy(osc_weights* w);

/* Buffer sizes for M activation rows (dense) or M_total rows in at most E expert segments (grouped). */
osc_status osc_act_sizes(const osc_weights* w, int M, osc_act_sizes_t* out);

/* Algorithm 2, fused: index lookup, back-up of the flagged channels into xo (the buffer B),
 * zero-out, CalculateScale, Quantize.  X: dev bf16 [M, ldx]. */
osc_status osc_quantize_extract(const osc_weights* w, const void* X, int M, int64_t ldx,
                                void* xq, void* sfa, void* xo, void* stream);

/* Eq. 5 on pre-quantized activations: block-scaled FP4 path and BF16 bypass path accumulate
 * into one fp32 tile; Y = bf16(acc).  Y: dev bf16 [M, ldy]. */
osc_status osc_gemm_dual(const osc_weights* w, const void* xq, const void* sfa, const void* xo, int M,
                         void* Y, int64_t ldy, void* stream);

/* osc_quantize_extract followed by osc_gemm_dual; workspace (dev) holds xq/sfa/xo between the two and is scratch: its
 * content after the call is unspecified.  With sixteen rows or fewer and a short K loop the few-row kernel quantizes
 * the activations of each CTA's K slice itself (the scales of Algorithm 2 are local to a group) and no quantizer
 * kernel runs; Y equals the two-step result bit for bit. */
osc_status osc_linear(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                      void* workspace, size_t workspace_bytes, void* stream);

/* osc_linear without a caller workspace.  (The paper has no counterpart: this is a deployment aid.)
 * For callers that cannot supply scratch memory - e.g. a plug-in whose host hands it only the input and
 * output pointers, or code that must not allocate because an allocation would synchronise the device.
 * The scratch between the two kernels lives in a fixed array of OSC_STATIC_SCRATCH_BYTES inside the
 * library (every GPU that loads the library holds it until the process exits).  The call allocates
 * nothing.  Limits and rules:
 *   - dense weights only; the workspace size osc_act_sizes reports for M must not exceed
 *     OSC_STATIC_SCRATCH_BYTES (e.g. M <= 1024 at K = 4096, K_o_pad = 256), else OSC_ERR_WORKSPACE;
 *   - the first call on each device looks the array's device address up (one runtime query, with
 *     that device current); make that first call before any stream capture;
 *   - all calls on a device share the one array: two calls that may overlap on the GPU (different
 *     streams without an ordering between them) race on it.  Calls on one stream are safe, and no call
 *     depends on what an earlier one left behind.
 * Arguments, layouts, status codes and asynchrony are those of osc_linear. */
#define OSC_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
osc_status osc_linear_static(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                             void* stream);

/* ---- RMSNorm fused in front of Algorithm 2 -----------------------------------------------------------
 * Section 3.3 places the OSC quantizer directly behind the operator that produces the activations; for the
 * QKV and gate/up projections of a decoder layer that operator is an RMSNorm.  These calls read the residual
 * stream H once and never write the normalized tensor:
 *
 *   r_m = fl32( 1 / sqrt( (1/K) sum_k H[m,k]^2 + eps ) ),   X[m,k] = bf16( fl32( fl32( H[m,k] * r_m ) * gamma[k] ) )
 *
 * the statistic in IEEE double (squares exact, the sum accumulated in double, division and square root in
 * double, then one rounding to fp32), the element-wise part as two fp32 multiplications and one rounding
 * (nearest, ties to even) to bf16; Algorithm 2 then runs on X as in osc_quantize_extract.
 *   H      dev bf16 [M, ldh] (ldh >= K, multiple of 8, 16-byte aligned); gamma dev bf16 [K], 16-byte aligned.
 *   K <= 8192 (a row is staged in shared memory), else OSC_ERR_SHAPE.  Dense weights only.
 * osc_rmsnorm writes X itself (dev bf16 [M, ldx]): the unfused reference point for tests and measurements.
 * osc_rmsnorm_quantize_extract's outputs equal osc_quantize_extract's on osc_rmsnorm's X bit for bit.
 * osc_rmsnorm_linear = osc_rmsnorm_quantize_extract + osc_gemm_dual through the workspace of osc_act_sizes.
 * Asynchronous on `stream`; status codes as above. */
osc_status osc_rmsnorm(const void* H, int M, int K, int64_t ldh, const void* gamma, float eps, void* X, int64_t ldx,
                       void* stream);
osc_status osc_rmsnorm_quantize_extract(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma,
                                        float eps, void* xq, void* sfa, void* xo, void* stream);
osc_status osc_rmsnorm_linear(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma, float eps,
                              void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream);

/* The same with the residual update of a decoder layer in front of the norm (Section 3.3: the quantizer sits
 * directly behind the operator that produces the activations; here that operator is "add, then RMSNorm"):
 *
 *   H'[m,k] = bf16( H[m,k] + R[m,k] )      one fp32 addition (exact, or past the bf16 rounding point), nearest even
 *
 * H' goes to Hout (dev bf16 [M, ldo]) and the norm and Algorithm 2 run on H'.  R: dev bf16 [M, ldr], the branch
 * output (attention or MLP) to add.  Hout may be H or R themselves (update in place); other overlaps are not
 * allowed.  ldr, ldo >= K, multiples of 8; R, Hout 16-byte aligned.  Everything else as in the calls above;
 * osc_add_rmsnorm is the unfused reference point and writes X as osc_rmsnorm does. */
osc_status osc_add_rmsnorm(const void* H, const void* R, int M, int K, int64_t ldh, int64_t ldr, const void* gamma, float eps,
                           void* Hout, int64_t ldo, void* X, int64_t ldx, void* stream);
osc_status osc_add_rmsnorm_quantize_extract(const osc_weights* w, const void* H, const void* R, int M, int64_t ldh,
                                            int64_t ldr, const void* gamma, float eps, void* Hout, int64_t ldo, void* xq,
                                            void* sfa, void* xo, void* stream);
osc_status osc_add_rmsnorm_linear(const osc_weights* w, const void* H, const void* R, int M, int64_t ldh, int64_t ldr,
                                  const void* gamma, float eps, void* Hout, int64_t ldo, void* Y, int64_t ldy,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* Grouped (MoE) form: rows of X_perm are sorted by expert, expert e owns rows
 * [off[e], off[e+1]); off: dev int32 [E+1], off[E] == M_total.  Expert e's scale rows start
 * at scale row sum_{e'<e} roundup(m_e', 128).  The tile schedule is built on the device. */
osc_status osc_linear_grouped(const osc_weights* w, const void* X_perm, const int32_t* off, int M_total,
                              int64_t ldx, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                              void* stream);

/* Grouped form with the dispatch fused behind the quantizer.  In a mixture-of-experts layer a token goes to several
 * experts and Algorithm 2 does not depend on the expert (one table per layer): X holds the T tokens once
 * (dev bf16 [T, ldx]), row_token (dev int32 [M_total]) names the source token of every permuted row, off as in
 * osc_linear_grouped.  The tokens are quantized once and their packed codes, scale bytes and backed-up channels are
 * copied to the rows their experts own; the result equals osc_linear_grouped on X_perm[r] = X[row_token[r]] bit for
 * bit, without X_perm ever existing.  Indices outside [0, T) are clamped.  The workspace holds the grouped buffers
 * of osc_act_sizes(w, M_total) followed by the T tokens' quantized form: ask osc_gather_workspace_bytes. */
osc_status osc_gather_workspace_bytes(const osc_weights* w, int T, int M_total, size_t* bytes);
osc_status osc_linear_grouped_gather(const osc_weights* w, const void* X, int T, int64_t ldx, const int32_t* row_token,
                                     const int32_t* off, int M_total, void* Y, int64_t ldy, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* The same behind an RMSNorm (the router's tokens come straight from the residual stream H, dev bf16 [T, ldh]):
 * osc_rmsnorm_quantize_extract's kernel on the T tokens, then the gather.  Equals osc_linear_grouped_gather on
 * osc_rmsnorm's output bit for bit; K <= 8192; workspace as above. */
osc_status osc_rmsnorm_linear_grouped_gather(const osc_weights* w, const void* H, int T, int64_t ldh, const void* gamma,
                                             float eps, const int32_t* row_token, const int32_t* off, int M_total, void* Y,
                                             int64_t ldy, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------- offline profiling */

/* Scratch bytes osc_profile_lut needs for a K-channel slice (an fp64 sum and 32 counters per group). */
osc_status osc_profile_scratch_bytes(int K, size_t* bytes);

/* Offline profiling of one (position, layer) slice of calibration activations (Section 2.1-2.2, Eq. 1-4, and
 * Algorithm 1 for that slice).  X: dev bf16 [S, ldx], S tokens, K channels, groups of 32.
 *   T_l = alpha * mean|X|                                    (Eq. 1; the paper uses alpha = 5)
 *   per token and group the first channel with the largest magnitude (Eq. 2) votes if that magnitude
 *   exceeds T_l (Eq. 3); per group lut[k] = the channel with most votes (smallest index among equals) or -1
 *   if no token voted (Algorithm 1), n_total[k] = votes, n_hit[k] = votes of the winner (Eq. 4: the clustering
 *   density is n_hit[k] / n_total[k]).
 * Outputs (dev): lut int8 [K/32], n_hit int32 [K/32], n_total int32 [K/32], threshold_bits uint32 [1] = bit
 * pattern of the largest bf16 magnitude <= T_l (for bf16 data |x| > T_l is exactly bits(|x|) > that pattern;
 * T_l itself is formed in fp64).  scratch: dev, zeroed by the call.  The resulting lut (copied to the host) is
 * what osc_prepare_weights takes with lut_c = 1. */
osc_status osc_profile_lut(const void* X, int S, int K, int64_t ldx, float alpha, void* scratch, size_t scratch_bytes,
                           void* lut, void* n_hit, void* n_total, void* threshold_bits, void* stream);

/* ------------------------------------------------------------- FP8 fallback */

typedef struct osc_fp8_weights osc_fp8_weights;

typedef struct {
    size_t x8_bytes;        /* M * K */
    size_t sx_bytes;        /* M * 4 */
    size_t sched_bytes;     /* grouped only */
    size_t x8_offset;       /* placement inside the workspace of osc_fp8_linear[_grouped] */
    size_t sx_offset;
    size_t sched_offset;
    size_t workspace_bytes;
} osc_fp8_act_sizes_t;

/* Section 3.4: the W2 / down-projection runs in FP8.  Offline: per output row n,
 * sw[n] = max(amax_n, 2^-40)/448 and w8 = E4M3(W * 448/max(amax_n, 2^-40)) (nearest-even, saturating).
 * w8: dev [E*N*K] bytes, sw: dev fp32 [E*N]. */
osc_status osc_fp8_prepare_weights(const void* W, int N, int K, int64_t ldw, void* w8, void* sw,
                                   void* stream, osc_fp8_weights** out);
osc_status osc_fp8_prepare_weights_grouped(const void* W, int E, int N, int K, void* w8, void* sw,
                                           void* stream, osc_fp8_weights** out);
osc_status osc_fp8_weights_destroy(osc_fp8_weights* w);
osc_status osc_fp8_act_sizes(const osc_fp8_weights* w, int M, osc_fp8_act_sizes_t* out);

/* Per-token dynamic E4M3 quantization: sx[m] and x8[m,:] as above, per activation row. */
osc_status osc_fp8_quantize(const void* X, int M, int K, int64_t ldx, void* x8, void* sx, void* stream);

/* Y[m,n] = bf16(sx[m] * sw[n] * sum_k x8[m,k] * w8[n,k]), fp32 accumulation. */
osc_status osc_fp8_gemm(const osc_fp8_weights* w, const void* x8, const void* sx, int M, void* Y,
                        int64_t ldy, void* stream);

osc_status osc_fp8_linear(const osc_fp8_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes, void* stream);

osc_status osc_fp8_linear_grouped(const osc_fp8_weights* w, const void* X_perm, const int32_t* off,
                                  int M_total, int64_t ldx, void* Y, int64_t ldy, void* workspace,
                                  size_t workspace_bytes, void* stream);

/* ---- SwiGLU fused in front of the per-token FP8 quantizer ---------------------------------------------
 * The producer of the down projection's input (Section 3.3 places the quantizer behind the operator that
 * produces the activations; Section 3.4 makes it FP8 for this input):
 *
 *   h[m,i] = bf16( silu(GU[m,i]) * GU[m,I+i] ),   silu(g) = g * (1 / (1 + exp32(-g)))
 *
 * in fp32, every step an IEEE operation (two multiplications and one reciprocal in silu): exp32(z) takes
 * t = z * log2(e) clamped to [-64, 126], n = rint(t), f = t - n, the degree-5 Taylor polynomial of 2^f by fused
 * multiply-adds, times 2^n.  The
 * per-token quantizer then works on the bf16 row h as osc_fp8_quantize does.
 *   GU  dev bf16 [M, ldg]: gate columns [0, I), up columns [I, 2I); ldg >= 2I, multiple of 8, 16-byte aligned.
 *   I   multiple of 128, <= 16384 (a row of h is held in registers), else OSC_ERR_SHAPE.
 * osc_swiglu writes h itself (dev bf16 [M, ldh]): the unfused reference point.  osc_swiglu_fp8_quantize's
 * outputs equal osc_fp8_quantize's on osc_swiglu's h bit for bit.  osc_swiglu_fp8_linear (dense weights with
 * K = I) = osc_swiglu_fp8_quantize + osc_fp8_gemm through the workspace of osc_fp8_act_sizes. */
osc_status osc_swiglu(const void* GU, int M, int I, int64_t ldg, void* H, int64_t ldh, void* stream);
osc_status osc_swiglu_fp8_quantize(const void* GU, int M, int I, int64_t ldg, void* x8, void* sx, void* stream);
osc_status osc_swiglu_fp8_linear(const osc_fp8_weights* w, const void* GU, int M, int64_t ldg, void* Y, int64_t ldy,
                                 void* workspace, size_t workspace_bytes, void* stream);
/* Grouped (MoE) form: rows of GU_perm (dev bf16 [M_total, ldg], the experts' gate|up outputs) sorted by expert as in
 * osc_fp8_linear_grouped; the per-token quantizer does not depend on the expert, so this is
 * osc_swiglu_fp8_quantize on all rows + the grouped FP8 GEMM.  Workspace: osc_fp8_act_sizes(w, M_total). */
osc_status osc_swiglu_fp8_linear_grouped(const osc_fp8_weights* w, const void* GU_perm, const int32_t* off, int M_total,
                                         int64_t ldg, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                         void* stream);

/* ---- SwiGLU in the epilogue of the gate|up projection ------------------------------------------------------
 * The next step of the same placement (Section 3.3): the activation is applied where the gate|up projection's
 * accumulators are, so the [M, 2I] output of that projection is never written or read; H [M, I] goes to the down
 * projection's FP8 quantizer (Section 3.4) at half the bytes.
 *   W    dev bf16 [2I, ldw]: gate rows [0, I) above up rows [I, 2I) (the nn.Linear layout of a fused gate_up weight).
 *   osc_gate_up_weight_sizes / osc_prepare_weights_gate_up: as osc_weight_sizes / osc_prepare_weights with N = 2I;
 *        meta is larger (a second per-tile copy of the weight scales, rows of a tile in gate|up order).  The handle
 *        is a full dense OSC handle: osc_linear, osc_gemm_dual, ... give the plain [M, 2I] projection with it.
 *   osc_linear_swiglu: H = bf16( silu(bf16(Yg)) * bf16(Yu) ) with Y = the OSC linear of Algorithm 2 + Eq. 5 and the
 *        activation arithmetic of osc_swiglu: bit for bit what osc_swiglu gives on osc_gemm_dual's output for the same
 *        quantized operands.  H dev bf16 [M, ldh], ldh >= I, multiple of 8.  I a multiple of 64.
 *        Workspace: osc_linear_swiglu_workspace_bytes(w, M) (the buffers of osc_act_sizes; problems of up to 256 rows
 *        run the plain projection into a scratch [M, 2I] behind them and the stand-alone activation).
 *   osc_rmsnorm_linear_swiglu: the same behind an RMSNorm fused into the quantizer (as osc_rmsnorm_linear).
 * Errors: OSC_ERR_INVALID_ARG for a handle not prepared by osc_prepare_weights_gate_up, otherwise as osc_linear. */
osc_status osc_gate_up_weight_sizes(int I, int K, const int8_t* lut, int lut_c, osc_weight_sizes_t* out);
osc_status osc_prepare_weights_gate_up(const void* W, int I, int K, int64_t ldw, const int8_t* lut, int lut_c, void* wq,
                                       void* sfw, void* wo, void* meta, void* stream, osc_weights** out);
osc_status osc_linear_swiglu_workspace_bytes(const osc_weights* w, int M, size_t* bytes);
osc_status osc_linear_swiglu(const osc_weights* w, const void* X, int M, int64_t ldx, void* H, int64_t ldh, void* workspace,
                             size_t workspace_bytes, void* stream);
osc_status osc_rmsnorm_linear_swiglu(const osc_weights* w, const void* Hin, int M, int64_t ldh_in, const void* gamma, float eps,
                                     void* H, int64_t ldh, void* workspace, size_t workspace_bytes, void* stream);
/* Grouped (MoE) forms: E experts' gate|up matrices stacked as W[E][2I][K]; one table for the layer.
 *   osc_gate_up_weight_sizes_grouped / osc_prepare_weights_gate_up_grouped: as osc_prepare_weights_grouped with N = 2I, meta
 *        additionally holding every expert's per-tile scale copy in gate|up order.  The handle also serves
 *        osc_linear_grouped and osc_linear_grouped_gather (the plain [M_total, 2I] projection).
 *   osc_linear_swiglu_grouped: rows of X_perm sorted by expert, off as in osc_linear_grouped; H dev bf16 [M_total, ldh].
 *        Workspace: osc_linear_swiglu_workspace_bytes(w, M_total).  Experts of fewer than 96 rows on average run the plain
 *        grouped projection into a scratch behind the workspace and the stand-alone activation.
 *   osc_linear_swiglu_grouped_gather / osc_rmsnorm_linear_swiglu_grouped_gather: the dispatch fused behind the quantizer
 *        (as osc_linear_grouped_gather / osc_rmsnorm_linear_grouped_gather); workspace: osc_swiglu_gather_workspace_bytes.
 *   Per expert the result equals the dense call on that expert's rows and weights: bit for bit where both run the CTA-pair
 *   kernel (experts of more than 256 rows in a layer of large experts), within the fp32 accumulation-order rounding otherwise. */
osc_status osc_gate_up_weight_sizes_grouped(int E, int I, int K, const int8_t* lut, int lut_c, osc_weight_sizes_t* out);
osc_status osc_prepare_weights_gate_up_grouped(const void* W, int E, int I, int K, const int8_t* lut, int lut_c, void* wq,
                                               void* sfw, void* wo, void* meta, void* stream, osc_weights** out);
osc_status osc_linear_swiglu_grouped(const osc_weights* w, const void* X_perm, const int32_t* off, int M_total, int64_t ldx,
                                     void* H, int64_t ldh, void* workspace, size_t workspace_bytes, void* stream);
osc_status osc_swiglu_gather_workspace_bytes(const osc_weights* w, int T, int M_total, size_t* bytes);
osc_status osc_linear_swiglu_grouped_gather(const osc_weights* w, const void* X, int T, int64_t ldx, const int32_t* row_token,
                                            const int32_t* off, int M_total, void* H, int64_t ldh, void* workspace,
                                            size_t workspace_bytes, void* stream);
osc_status osc_rmsnorm_linear_swiglu_grouped_gather(const osc_weights* w, const void* Hin, int T, int64_t ldh_in, const void* gamma,
                                                    float eps, const int32_t* row_token, const int32_t* off, int M_total, void* H,
                                                    int64_t ldh, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------- MXFP8 form of the fallback (Section 3.4) */

/* Section 3.4 allows "FP8 (or equivalent 8-bit micro-scaling formats)" for the W2 inputs and Section 4
 * ("Implementation Details") states that the experiments fall back to MXFP8.  This group of calls is that
 * form: E4M3 elements with one E8M0 scale per 32 channels along K (OCP MX v1.0: scale =
 * 2^(floor(log2 amax) - 8), i.e. code = max(biased exponent of amax - 8, 0); elements rounded to nearest
 * even, saturating at 448), for activations (online) and weights (offline) alike, no channel extracted.
 * Scales use the same 128 x 4 block layout as the MXFP4 scales (see osc_quantize_extract):
 * ceil(rows/128) * (K/128) * 512 bytes; bytes of rows past the end are written as 0.
 * Dense and grouped (MoE) problems; the grouped calls follow osc_fp8_linear_grouped (rows sorted by expert,
 * device-resident offsets, every expert's activation scales starting on a 128-row scale block, weights stacked
 * [E, N, K] with per-expert scale blocks).  Same conventions as the other calls: device pointers,
 * 16-byte alignment, leading dimensions in elements and multiples of 8, asynchronous on `stream`,
 * no allocation, M == 0 is a successful no-op, K % 128 == 0, N % 64 == 0. */
typedef struct osc_mxfp8_weights osc_mxfp8_weights;

typedef struct {
    size_t w8_bytes;        /* E * N * K */
    size_t sfw_bytes;       /* E * ceil(N/128) * (K/128) * 512 */
} osc_mxfp8_weight_sizes_t;

typedef struct {
    size_t x8_bytes;        /* M * K */
    size_t sfa_bytes;       /* ceil(M/128) * (K/128) * 512; grouped: (M/128 + E) row blocks */
    size_t sched_bytes;     /* grouped only */
    size_t x8_offset;       /* placement inside the workspace of osc_mxfp8_linear[_grouped] */
    size_t sfa_offset;
    size_t sched_offset;
    size_t workspace_bytes;
} osc_mxfp8_act_sizes_t;

osc_status osc_mxfp8_weight_sizes(int E, int N, int K, osc_mxfp8_weight_sizes_t* out);

/* Offline: w8 [N,K] E4M3 bytes and sfw (block layout) from W (dev bf16 [N, ldw]).  The handle borrows
 * w8 and sfw, which must outlive it; the caller owns every buffer. */
osc_status osc_mxfp8_prepare_weights(const void* W, int N, int K, int64_t ldw, void* w8, void* sfw, void* stream,
                                     osc_mxfp8_weights** out);
osc_status osc_mxfp8_prepare_weights_grouped(const void* W, int E, int N, int K, void* w8, void* sfw, void* stream,
                                             osc_mxfp8_weights** out);
osc_status osc_mxfp8_weights_destroy(osc_mxfp8_weights* w);
osc_status osc_mxfp8_act_sizes(const osc_mxfp8_weights* w, int M, osc_mxfp8_act_sizes_t* out);

/* Online: x8 [M,K] bytes and sfa (block layout) from X (dev bf16 [M, ldx]). */
osc_status osc_mxfp8_quantize(const void* X, int M, int K, int64_t ldx, void* x8, void* sfa, void* stream);

/* Y[m,n] = bf16(sum_g 2^(sfa[m,g]-127) 2^(sfw[n,g]-127) sum_{k in g} x8[m,k] w8[n,k]), fp32 accumulation
 * on the block-scaled tensor-core path. */
osc_status osc_mxfp8_gemm(const osc_mxfp8_weights* w, const void* x8, const void* sfa, int M, void* Y, int64_t ldy,
                          void* stream);

/* quantize + gemm through a caller-provided workspace of at least osc_mxfp8_act_sizes().workspace_bytes. */
osc_status osc_mxfp8_linear(const osc_mxfp8_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* stream);
osc_status osc_mxfp8_linear_grouped(const osc_mxfp8_weights* w, const void* X_perm, const int32_t* off, int M_total,
                                    int64_t ldx, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                    void* stream);

/* ------------------- dynamic-protection control group (Section 4.2), a baseline */

/* The paper compares OSC with an "idealized Dynamic Protection baseline": per token and per 32-group the
 * element of largest magnitude is detected at run time, kept in high precision and removed before the group
 * is scaled and quantized.  These calls are that baseline, built so that its cost can be measured beside
 * osc_linear on the same shapes (Section 4.2, "Hardware-Efficiency Trade-offs").  Because any channel can be
 * picked by some token, the weights are MXFP4 of the WHOLE matrix (no column zeroed) plus the bf16 matrix
 * itself as the high-precision operand; the extracted elements are handed to the tensor cores as a dense
 * [M, K] bf16 matrix xo that is +0 except at the extracted positions (one non-zero per 32 channels), so the
 * high-precision branch of Eq. 5 runs over all K channels instead of K_o.  The handle is an osc_weights with
 * K_o = K_o_pad = K; it is accepted by osc_gemm_dual, osc_weights_destroy and the osc_dyn_* calls only.
 * Dense problems only.  osc_dyn_weight_sizes fills the same struct as osc_weight_sizes (wo_bytes = N*K*2). */
typedef struct {
    size_t xq_bytes, sfa_bytes;     /* as osc_act_sizes */
    size_t xo_bytes;                /* M * K * 2: the dense high-precision operand */
    size_t idx_bytes;               /* M * K/32: local channel 0..31 of the extracted element, uint8 */
    size_t val_bytes;               /* M * K/32 * 2: the extracted elements, bf16 bit copies */
    size_t xq_offset, sfa_offset, xo_offset, idx_offset, val_offset;
    size_t workspace_bytes;
} osc_dyn_act_sizes_t;

osc_status osc_dyn_weight_sizes(int N, int K, osc_weight_sizes_t* out);
osc_status osc_dyn_prepare_weights(const void* W, int N, int K, int64_t ldw, void* wq, void* sfw, void* wo, void* meta,
                                   void* stream, osc_weights** out);
osc_status osc_dyn_act_sizes(const osc_weights* w, int M, osc_dyn_act_sizes_t* out);

/* Run-time extraction + MXFP4 of the rest.  Ties between equal magnitudes take the lowest channel; an all-zero
 * group extracts its first element.  xq, sfa as osc_quantize_extract; xo, idx, val as described above. */
osc_status osc_dyn_quantize_extract(const osc_weights* w, const void* X, int M, int64_t ldx, void* xq, void* sfa,
                                    void* xo, void* idx, void* val, void* stream);

/* osc_dyn_quantize_extract + the dual-path GEMM with K_o = K. */
osc_status osc_dyn_linear(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes, void* stream);

/* --------------------------------------------- NVFP4 / G = 16 variant of the OSC path */

/* The paper reports OSC on NVFP4 too (efficiency table, row G = 16; Section 5) without stating the arithmetic.
 * These calls are the reading taken here: E2M1 elements in blocks of 16 along K, one unsigned E4M3 scale per
 * block, and a tensor-level scale restricted to a power of two (2^ex for the activations, 2^ew for the weights,
 * chosen by the caller, e.g. the smallest e with amax * 2^-e <= 6 * 448), so that the high-precision branch
 * lives in the same scaled domain exactly and both paths share one accumulator:
 *   x' = x * 2^-e;  per block, after the flagged channels are backed up (as bf16(x')) and zeroed:
 *   t = fl32(amax' * fl32(1/6)), scale byte = E4M3(t) (nearest even, saturating),
 *   codes = E2M1(fl32(x' * fl32(1/scale))) (sign-only zeros when the scale is zero);
 *   Y = bf16( 2^(ex+ew) * ( sum_b sa*sw * sum_{k in b} xq*wq  +  sum_t xo*wo ) ).
 * The table lists local channels 0..15 per 16-channel group: lut16 is host int8 [K/16][lut_c], -1 = none.
 * Scale bytes: 512-byte blocks of 128 rows x 64 channels,
 *   byte(r, b) = ((r/128)*(K/64) + b/4)*512 + (r%32)*16 + ((r%128)/32)*4 + b%4   (b = block index along K),
 * ceil(rows/128) * (K/64) * 512 bytes per tensor.  Same conventions as osc_linear; the grouped form follows below.
 * The handle is an osc_weights accepted only by the osc_nvfp4_* calls and osc_weights_destroy;
 * osc_nvfp4_weight_sizes and osc_nvfp4_act_sizes fill the structs of their MXFP4 counterparts. */
osc_status osc_nvfp4_weight_sizes(int N, int K, const int8_t* lut16, int lut_c, osc_weight_sizes_t* out);
osc_status osc_nvfp4_prepare_weights(const void* W, int N, int K, int64_t ldw, const int8_t* lut16, int lut_c, int ew,
                                     void* wq, void* sfw, void* wo, void* meta, void* stream, osc_weights** out);
osc_status osc_nvfp4_act_sizes(const osc_weights* w, int M, osc_act_sizes_t* out);
osc_status osc_nvfp4_quantize_extract(const osc_weights* w, const void* X, int M, int64_t ldx, int ex, void* xq,
                                      void* sfa, void* xo, void* stream);
osc_status osc_nvfp4_gemm(const osc_weights* w, const void* xq, const void* sfa, const void* xo, int M, int ex, void* Y,
                          int64_t ldy, void* stream);
osc_status osc_nvfp4_linear(const osc_weights* w, const void* X, int M, int64_t ldx, int ex, void* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Grouped (MoE) form of the NVFP4 path: E experts stacked as W[E][N][K] (ldw = K), one table and one weight
 * tensor exponent ew for the layer, every expert quantized on its own (its scale blocks start on a 128-row
 * block); buffers are E times the dense sizes (osc_nvfp4_weight_sizes_grouped).  Rows of X_perm sorted by
 * expert and off as in osc_linear_grouped; expert e's activation scale rows start at scale row
 * sum_{e'<e} roundup(m_e', 128); workspace from osc_nvfp4_act_sizes(w, M_total).  A grouped handle is accepted
 * by osc_nvfp4_act_sizes, osc_nvfp4_linear_grouped, the two gathered forms below and osc_weights_destroy only. */
osc_status osc_nvfp4_weight_sizes_grouped(int E, int N, int K, const int8_t* lut16, int lut_c, osc_weight_sizes_t* out);
osc_status osc_nvfp4_prepare_weights_grouped(const void* W, int E, int N, int K, const int8_t* lut16, int lut_c, int ew,
                                             void* wq, void* sfw, void* wo, void* meta, void* stream, osc_weights** out);
osc_status osc_nvfp4_linear_grouped(const osc_weights* w, const void* X_perm, const int32_t* off, int M_total, int64_t ldx,
                                    int ex, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream);

/* The producer fusion and the dispatch gather in the NVFP4 / G = 16 form (Section 3.3 places the quantizer behind
 * the operator that produces the activations; the efficiency table's G = 16 row is this format).
 * osc_nvfp4_rmsnorm_quantize_extract: RMSNorm (arithmetic as osc_rmsnorm) and the NVFP4 form of Algorithm 2 in one
 *   pass over H (dev bf16 [M, ldh], K <= 8192); ex is the tensor exponent of the NORMALIZED activations; outputs as
 *   osc_nvfp4_quantize_extract writes them, bit for bit what that call gives on osc_rmsnorm's output.
 * osc_nvfp4_rmsnorm_linear = that + osc_nvfp4_gemm, workspace from osc_nvfp4_act_sizes.
 * osc_nvfp4_linear_grouped_gather / osc_nvfp4_rmsnorm_linear_grouped_gather: as osc_linear_grouped_gather /
 *   osc_rmsnorm_linear_grouped_gather with a grouped NVFP4 handle: the T tokens are quantized once (scale blocks of
 *   64 channels) and their quantized rows copied to the rows their experts own; equals osc_nvfp4_linear_grouped on
 *   X_perm[r] = X[row_token[r]] bit for bit.  Workspace: osc_nvfp4_gather_workspace_bytes.
 * Errors as for their MXFP4 counterparts. */
osc_status osc_nvfp4_rmsnorm_quantize_extract(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma,
                                              float eps, int ex, void* xq, void* sfa, void* xo, void* stream);
osc_status osc_nvfp4_rmsnorm_linear(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma, float eps,
                                    int ex, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream);
osc_status osc_nvfp4_gather_workspace_bytes(const osc_weights* w, int T, int M_total, size_t* bytes);
osc_status osc_nvfp4_linear_grouped_gather(const osc_weights* w, const void* X, int T, int64_t ldx, const int32_t* row_token,
                                           const int32_t* off, int M_total, int ex, void* Y, int64_t ldy, void* workspace,
                                           size_t workspace_bytes, void* stream);
osc_status osc_nvfp4_rmsnorm_linear_grouped_gather(const osc_weights* w, const void* H, int T, int64_t ldh, const void* gamma,
                                                   float eps, const int32_t* row_token, const int32_t* off, int M_total, int ex,
                                                   void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OSC_H_ */
