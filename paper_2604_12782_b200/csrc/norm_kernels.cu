// Producers fused with the quantizer that follows them: RMSNorm + Algorithm 2 (below), SwiGLU + per-token FP8 (end of file).
//
// RMSNorm fused in front of Algorithm 2 (Section 3.3 puts the OSC quantizer directly behind the operator that
// produces the activations; in a decoder layer that operator is the RMSNorm in front of the QKV and gate/up
// projections).  One pass over the residual stream instead of three (norm read + norm write + quantizer read).
//
// Arithmetic (statistics in double, element-wise part in fp32, one rounding to bf16):
//   r   = fl32( 1 / sqrt( (1/K) sum_k x_k^2 + eps ) )     squares and sum in double (squares of bf16 are exact)
//   y_k = bf16( fl32( fl32(x_k * r) * gamma_k ) )
// followed by Algorithm 2 on the bf16 row y exactly as quant_extract_kernel does it (back-up of the flagged
// channels, zero-out, E8M0 scale per 32, E2M1 codes).  The sum is a fixed tree (two partial sums per lane,
// butterfly over the warp), so results are deterministic; against the exactly rounded sum it is off by a few
// units of the 53rd bit, which changes r only if 1/sqrt(..) lies within ~1e-16 of an fp32 rounding boundary.
//
// Two warps per row (K <= 8192; named barriers keep the pair in step): one lane fetches the row into shared memory
// with one bulk copy (cp.async.bulk, one mbarrier per row); the first pass sums the squares; the second normalizes the row in place (bf16); then the
// flagged channels are copied out through the channel list (lane t takes list entry t: 64-byte coalesced stores
// into xo) and zeroed in the shared row; last, every lane quantizes whole 32-channel groups as in
// quant_extract_kernel (amax without shuffles, one 16-byte store of codes, the four scale bytes of a 128-channel
// block gathered by two shuffles).  Handling the flagged channels in registers, lane by lane through the bit mask,
// made the lanes of a warp diverge at nearly every word (22 of 32 threads active on average, twice the
// instructions).  A first version did the element-wise part in double too, with the
// bf16 <-> double conversions as integer operations: ~90 instructions per element, the unrolled row loop no
// longer fit the instruction cache, 172 us for 8192 x 4096 (ALU pipe and instruction fetch, fp64 pipe at 3 %).
// Holding the row in registers needs the row loop fully unrolled, which made the compiler hoist every load of the
// second pass and spill.
#include "common.cuh"

namespace osc {

constexpr int RN_ROWS = 14;    // rows per CTA (28 rows in flight per SM: 8 KB of shared memory per row at K = 4096)
constexpr int RN_WPR = 2;      // warps per row: twice the warps to hide latency with, for the same shared memory
constexpr int RN_TEAM = 32 * RN_WPR;
constexpr int RN_THREADS = RN_ROWS * RN_TEAM;

// barrier of the two warps of a row (named barriers 1..RN_ROWS; 0 is the CTA's)
__device__ __forceinline__ void team_sync(int slot) {
    asm volatile("bar.sync %0, %1;" ::"r"(slot + 1), "r"(RN_TEAM) : "memory");
}

// Two CTAs per SM (28 rows in flight) need at most 36 registers per thread; the residual update is a template
// parameter so that the plain form keeps its 32.
// FMT: FMT_MXFP4 (Algorithm 2 as stated) or FMT_NVFP4 (blocks of 16 with E4M3 scales, tensor scale 2^tensor_e,
// scale blocks of 64 channels; fp32 scale arithmetic, so one CTA per SM).
template <bool QUANT, bool ADD, int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(RN_THREADS, FMT == FMT_MXFP4 ? 2 : 1)
rmsnorm_quant_kernel(const uint16_t* __restrict__ H, int64_t ldh, int M, int M_pad, int K,
                     const uint16_t* __restrict__ gamma, float eps, uint16_t* __restrict__ Xn, int64_t ldx,
                     const int32_t* __restrict__ idx_o, uint8_t* __restrict__ xq,
                     uint8_t* __restrict__ sf, uint16_t* __restrict__ xo, int Ko, int Kop,
                     const uint16_t* R, int64_t ldr, uint16_t* Hout, int64_t ldo, int tensor_e) {
    // [RN_ROWS][K / 8] rows, then per row: one mbarrier, two partial sums (double), one give-up flag
    extern __shared__ uint4 rn_rows[];
    grid_launch_dependents();
    const int slot = threadIdx.x / RN_TEAM;          // my row inside the CTA
    const int tl = threadIdx.x % RN_TEAM;            // my lane inside the row's team of two warps
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * RN_ROWS + slot;
    if (r >= M_pad) return;                          // both warps of a team take every exit together
    const int katoms = K / (FMT == FMT_NVFP4 ? 64 : 128);   // scale blocks along K
    // scale word of (row r, scale block a): block (r/128)*katoms + a, word (r%32)*4 + (r%128)/32
    uint32_t* sf_row = QUANT ? reinterpret_cast<uint32_t*>(sf + (size_t)(r / 128) * katoms * 512) + (r & 31) * 4 + ((r & 127) >> 5)
                             : nullptr;
    if (r >= M) {   // rows that only pad the last 128-row scale block
        grid_dependency_wait();
        if (QUANT)
            for (int a = tl; a < katoms; a += RN_TEAM) sf_row[(size_t)a * 128] = 0u;
        return;
    }
    const uint4* hrow = reinterpret_cast<const uint4*>(H + (int64_t)r * ldh);
    const uint4* grow = reinterpret_cast<const uint4*>(gamma);
    const int nch = K / 8;   // 16-byte chunks in the row

    uint4* row = rn_rows + (size_t)slot * nch;
    uint8_t* tail = reinterpret_cast<uint8_t*>(rn_rows + (size_t)RN_ROWS * nch);
    uint64_t* bar = reinterpret_cast<uint64_t*>(tail) + slot;
    double* part = reinterpret_cast<double*>(tail + RN_ROWS * 8) + slot * RN_WPR;
    volatile int* give_up = reinterpret_cast<volatile int*>(tail + RN_ROWS * 8 + RN_ROWS * RN_WPR * 8) + slot;
    if (tl == 0) {
        *give_up = 0;
        mbar_init(bar, 1);
        fence_barrier_init();
    }
    team_sync(slot);
    grid_dependency_wait();   // H may come from, and the outputs may still be read by, earlier kernels
    if (tl == 0) {
        mbar_arrive_expect_tx(bar, (uint32_t)K * 2u);
        bulk_load(row, hrow, (uint32_t)K * 2u, bar);
    }
    // a wait that gives up has recorded it in the device status word; the team carries on (with whatever the row
    // buffer holds) so that its barriers below stay matched
    wait_bounded(bar, 0u, give_up, 41);

    // ---- first pass: sum of squares, each warp over every second step of chunks.  With a residual update (R != null)
    // the row becomes h' = bf16(h + r) first - one fp32 addition, exact or beyond the bf16 rounding point, then nearest
    // even - which goes back to the residual stream (Hout; it may be H or R themselves: the row of H is already in
    // shared memory, and a chunk of R is read by the thread that then overwrites it) and replaces the shared row.
    const uint4* rrow = ADD ? reinterpret_cast<const uint4*>(R + (int64_t)r * ldr) : nullptr;
    uint4* orow = ADD ? reinterpret_cast<uint4*>(Hout + (int64_t)r * ldo) : nullptr;
    const int nsteps = (nch + RN_TEAM - 1) / RN_TEAM;
    double ss0 = 0.0, ss1 = 0.0, ss2 = 0.0, ss3 = 0.0;   // four chains: the fp64 pipe's latency is long
#pragma unroll 4
    for (int i = 0; i < nsteps; ++i) {
        const int c = i * RN_TEAM + tl;
        const uint4 v = (c < nch) ? row[c] : make_uint4(0u, 0u, 0u, 0u);
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
        if (ADD && c < nch) {
            const uint4 d = rrow[c];
            const uint32_t dw[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w[j] = bf162_bits(__floats2bfloat162_rn(__fadd_rn(__uint_as_float(w[j] << 16), __uint_as_float(dw[j] << 16)),
                                                        __fadd_rn(__uint_as_float(w[j] & 0xFFFF0000u), __uint_as_float(dw[j] & 0xFFFF0000u))));
            const uint4 hs = make_uint4(w[0], w[1], w[2], w[3]);
            row[c] = hs;
            orow[c] = hs;
        }
#pragma unroll
        for (int j = 0; j < 4; j += 2) {
            const double a0 = (double)__uint_as_float(w[j] << 16), b0 = (double)__uint_as_float(w[j] & 0xFFFF0000u);
            const double a1 = (double)__uint_as_float(w[j + 1] << 16), b1 = (double)__uint_as_float(w[j + 1] & 0xFFFF0000u);
            ss0 = fma(a0, a0, ss0);
            ss1 = fma(b0, b0, ss1);
            ss2 = fma(a1, a1, ss2);
            ss3 = fma(b1, b1, ss3);
        }
    }
    double ss = (ss0 + ss1) + (ss2 + ss3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    if (lane == 0) part[tl >> 5] = ss;
    team_sync(slot);
    ss = part[0] + part[1];   // the same two values in the same order in every lane of the team
    const float r32 = (float)(1.0 / sqrt(ss / (double)K + (double)eps));

    // ---- second pass: normalize; QUANT: in place in shared memory, else straight to global memory
#pragma unroll 4
    for (int i = 0; i < nsteps; ++i) {
        const int c = i * RN_TEAM + tl;
        if (c >= nch) break;
        const uint4 g4 = grow[c], v = row[c];
        const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w};
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float lo = __fmul_rn(__fmul_rn(__uint_as_float(w[j] << 16), r32), __uint_as_float(gw[j] << 16));
            const float hi = __fmul_rn(__fmul_rn(__uint_as_float(w[j] & 0xFFFF0000u), r32), __uint_as_float(gw[j] & 0xFFFF0000u));
            w[j] = bf162_bits(__floats2bfloat162_rn(lo, hi));   // nearest even; lo in the low half
        }
        if (QUANT) row[c] = make_uint4(w[0], w[1], w[2], w[3]);
        else *reinterpret_cast<uint4*>(Xn + (int64_t)r * ldx + c * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (!QUANT) return;
    team_sync(slot);

    // ---- Algorithm 2 on the normalized row.  Back-up and zero-out: entry t of the (ascending) channel list goes to
    // column t of xo; pad columns +0
    uint16_t* row16 = reinterpret_cast<uint16_t*>(row);
    for (int t = tl; t < Kop; t += RN_TEAM) {
        uint16_t e = 0;
        if (t < Ko) {
            const int ch = idx_o[t];
            e = row16[ch];
            row16[ch] = 0;
            if (FMT == FMT_NVFP4) e = nvfp4_backup(e, tensor_e);
        }
        xo[(int64_t)r * Kop + t] = e;
    }
    team_sync(slot);

    // every lane quantizes whole 32-channel groups
    const int ngrp = K / 32;
    for (int g0 = 0; g0 < ngrp; g0 += RN_TEAM) {
        const int g = g0 + tl;
        const bool in = g < ngrp;   // ngrp is a multiple of 4, so the four lanes of a scale word are in or out together
        uint32_t w[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint4 v = in ? row[4 * g + j] : make_uint4(0u, 0u, 0u, 0u);
            w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
        }
        if (FMT == FMT_NVFP4) {
            uint32_t q[4];
            const uint32_t codes = nvfp4_group(w, __uint_as_float((uint32_t)(127 - tensor_e) << 23), q);
            if (in) *reinterpret_cast<uint4*>(xq + (int64_t)r * (K / 2) + g * 16) = make_uint4(q[0], q[1], q[2], q[3]);
            // a 64-channel scale block is two 32-channel groups: two bytes from each of two neighbouring lanes
            uint32_t word = codes << (16 * (g & 1));
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
            if ((g & 1) == 0 && in) sf_row[(size_t)(g >> 1) * 128] = word;
            continue;
        }
        __nv_bfloat162 m2 = __habs2(as_bf162(w[0]));
#pragma unroll
        for (int t = 1; t < 16; ++t) m2 = __hmax2(m2, __habs2(as_bf162(w[t])));
        const uint32_t am2 = bf162_bits(m2);
        const uint32_t am = max(am2 & 0xFFFFu, am2 >> 16);
        // CalculateScale: E8M0 code = biased exponent of amax - 2, floored at 0; Quantize: exact power-of-two
        // scaling, hardware E2M1 rounding (nearest even, saturating)
        const int ex = (int)(am >> 7);
        int code = max(ex - 2, 0);
        if (ex == 255) code = 255;
        const __nv_bfloat162 inv2 = as_bf162(((uint32_t)(254 - min(code, 253)) << 7) * 0x10001u);
        uint32_t q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float f[8];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const uint32_t p = bf162_bits(__hmul2(as_bf162(w[4 * j + t]), inv2));
                f[2 * t] = __uint_as_float(p << 16);
                f[2 * t + 1] = __uint_as_float(p & 0xFFFF0000u);
            }
            q[j] = e2m1x8(f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
        }
        if (in) *reinterpret_cast<uint4*>(xq + (int64_t)r * (K / 2) + g * 16) = make_uint4(q[0], q[1], q[2], q[3]);
        // the four scale bytes of a 128-channel block are one 32-bit word: gather from the four lanes that hold them
        uint32_t word = (uint32_t)code << (8 * (g & 3));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        if ((g & 3) == 0 && in) sf_row[(size_t)(g >> 2) * 128] = word;
    }
}

constexpr int kRnTail = RN_ROWS * (8 + RN_WPR * 8 + 4) + 8;   // mbarriers, partial sums, give-up flags

template <bool QUANT, bool ADD, int FMT = FMT_MXFP4>
static cudaError_t launch_rmsnorm_cfg(dim3 grid, dim3 block, size_t smem, cudaStream_t st, const void* H, int64_t ldh, int M,
                                      int M_pad, int K, const void* gamma, float eps, void* Xn, int64_t ldx,
                                      const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko, int Kop, const void* R,
                                      int64_t ldr, void* Hout, int64_t ldo, int tensor_e = 0) {
    static PerDevice configured;
    if (cudaError_t e = opt_in_shared_memory(configured, rmsnorm_quant_kernel<QUANT, ADD, FMT>, RN_ROWS * 8192 * 2 + kRnTail)) return e;
    return launch_pdl(rmsnorm_quant_kernel<QUANT, ADD, FMT>, grid, block, smem, st, static_cast<const uint16_t*>(H), ldh, M, M_pad, K,
                      static_cast<const uint16_t*>(gamma), eps, static_cast<uint16_t*>(Xn), ldx, idx_o,
                      static_cast<uint8_t*>(xq), static_cast<uint8_t*>(sf), static_cast<uint16_t*>(xo), Ko, Kop,
                      static_cast<const uint16_t*>(R), ldr, static_cast<uint16_t*>(Hout), ldo, tensor_e);
}

// RMSNorm + the NVFP4 form of Algorithm 2 (no residual update in this form)
cudaError_t launch_rmsnorm_quant_nvfp4(const void* H, int64_t ldh, int M, int K, const void* gamma, float eps,
                                       const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko, int Kop, int tensor_e,
                                       cudaStream_t st) {
    if (M <= 0) return cudaSuccess;
    const int M_pad = (M + 127) / 128 * 128;
    const dim3 grid((M_pad + RN_ROWS - 1) / RN_ROWS), block(RN_THREADS);
    return launch_rmsnorm_cfg<true, false, FMT_NVFP4>(grid, block, (size_t)RN_ROWS * K * 2 + kRnTail, st, H, ldh, M, M_pad, K,
                                                      gamma, eps, nullptr, 0, idx_o, xq, sf, xo, Ko, Kop, nullptr, 0, nullptr, 0,
                                                      tensor_e);
}

// QUANT: Xn unused.  !QUANT: the quantizer arguments unused.  K <= 8192.  R != null: residual update h' = bf16(h + r)
// written to Hout before the norm.
cudaError_t launch_rmsnorm_quant(bool quant, const void* H, int64_t ldh, int M, int K, const void* gamma, float eps,
                                 void* Xn, int64_t ldx, const int32_t* idx_o, void* xq, void* sf,
                                 void* xo, int Ko, int Kop, cudaStream_t st, const void* R, int64_t ldr, void* Hout,
                                 int64_t ldo) {
    if (M <= 0) return cudaSuccess;
    const int M_pad = quant ? (M + 127) / 128 * 128 : M;
    const dim3 grid((M_pad + RN_ROWS - 1) / RN_ROWS), block(RN_THREADS);
    const size_t smem = (size_t)RN_ROWS * K * 2 + kRnTail;
    return quant ? (R ? launch_rmsnorm_cfg<true, true>(grid, block, smem, st, H, ldh, M, M_pad, K, gamma, eps, Xn, ldx, idx_o, xq, sf, xo, Ko, Kop, R, ldr, Hout, ldo)
                      : launch_rmsnorm_cfg<true, false>(grid, block, smem, st, H, ldh, M, M_pad, K, gamma, eps, Xn, ldx, idx_o, xq, sf, xo, Ko, Kop, R, ldr, Hout, ldo))
                 : (R ? launch_rmsnorm_cfg<false, true>(grid, block, smem, st, H, ldh, M, M_pad, K, gamma, eps, Xn, ldx, idx_o, xq, sf, xo, Ko, Kop, R, ldr, Hout, ldo)
                      : launch_rmsnorm_cfg<false, false>(grid, block, smem, st, H, ldh, M, M_pad, K, gamma, eps, Xn, ldx, idx_o, xq, sf, xo, Ko, Kop, R, ldr, Hout, ldo));
}

// ------------------------------------------------------------------ SwiGLU + per-token FP8
// The producer of the down projection's input fused with its quantizer (Section 3.3 puts the quantizer behind the
// producing operator; Section 3.4 makes it FP8 for this input): h = bf16(silu(gate) * up) is never written, the row
// goes from the gate/up projection's output straight to E4M3 codes and a per-row scale.  Arithmetic (fp32, every
// step an IEEE operation, so the codes are decided on identical values on every implementation):
//   exp32(z): t = z * log2(e) clamped to [-64, 126]; n = rint(t), f = t - n, p = degree-5 Taylor polynomial of 2^f
//             by fused multiply-adds, e = p * 2^n
//   silu(g) = g * (1 / (1 + exp32(-g)));  h = bf16(silu(g) * u)
// then amax' = max(amax, 2^-40), scale = amax'/448, codes = E4M3(h * (448/amax')) as in fp8_quant_kernel.
// One CTA per row, the bf16 row h held in registers between the amax pass and the encode pass (I <= 16384).
// The kernel is bound by instruction issue (ncu: issue slots 76 % busy at 47 instructions per element in a first
// version with three range checks, a full division and a degree-6 polynomial), which is why the arithmetic above
// is as lean as a reproducible definition allows.
__device__ __forceinline__ float exp32(float z) {
    const float t = fminf(fmaxf(__fmul_rn(z, 1.44269502f), -64.0f), 126.0f);   // NaN -> -64 (g itself carries the NaN on)
    // n = rint(t), nearest with ties to even: adding 1.5 * 2^23 rounds t to an integer in the last mantissa bits
    // (|t| < 2^22), and the integer can be read off the bit pattern; two additions instead of two conversions,
    // which run at a quarter of the rate
    const float tn = __fadd_rn(t, 12582912.0f);
    const float n = __fsub_rn(tn, 12582912.0f);
    const int ni = __float_as_int(tn) - 0x4B400000;
    const float f = __fsub_rn(t, n);
    float p = 0.00133335579f;
    p = __fmaf_rn(p, f, 0.00961812865f);
    p = __fmaf_rn(p, f, 0.0555041097f);
    p = __fmaf_rn(p, f, 0.240226507f);
    p = __fmaf_rn(p, f, 0.693147182f);
    p = __fmaf_rn(p, f, 1.0f);
    return __fmul_rn(p, __int_as_float((ni + 127) << 23));   // exact: -64 <= n <= 126 and p < 1.5
}
__device__ __forceinline__ float swiglu32(float g, float u) {
    const float d = __fadd_rn(1.0f, exp32(-g));
    return __fmul_rn(__fmul_rn(g, __frcp_rn(d)), u);
}
// The same two elements at a time on the packed fp32 instructions of sm_100 (add / mul / fma on register pairs, each
// half rounded to nearest like the scalar instruction): identical results, about a third fewer issue slots in a kernel
// that is bound by them.  exp32x2 takes g and computes exp32(-g): fl(g * -log2e) = fl(-g * log2e), and t - n is
// written as the fused n * -1 + t, whose product is exact.
__device__ __forceinline__ float2 exp32x2_neg(float2 g) {
    float2 t = __fmul2_rn(g, make_float2(-1.44269502f, -1.44269502f));
    t.x = fminf(fmaxf(t.x, -64.0f), 126.0f);
    t.y = fminf(fmaxf(t.y, -64.0f), 126.0f);
    const float2 tn = __fadd2_rn(t, make_float2(12582912.0f, 12582912.0f));
    const float2 n = __fadd2_rn(tn, make_float2(-12582912.0f, -12582912.0f));
    const int nx = __float_as_int(tn.x) - 0x4B400000, ny = __float_as_int(tn.y) - 0x4B400000;
    const float2 f = __ffma2_rn(n, make_float2(-1.0f, -1.0f), t);
    float2 p = make_float2(0.00133335579f, 0.00133335579f);
    p = __ffma2_rn(p, f, make_float2(0.00961812865f, 0.00961812865f));
    p = __ffma2_rn(p, f, make_float2(0.0555041097f, 0.0555041097f));
    p = __ffma2_rn(p, f, make_float2(0.240226507f, 0.240226507f));
    p = __ffma2_rn(p, f, make_float2(0.693147182f, 0.693147182f));
    p = __ffma2_rn(p, f, make_float2(1.0f, 1.0f));
    return __fmul2_rn(p, make_float2(__int_as_float((nx + 127) << 23), __int_as_float((ny + 127) << 23)));
}
__device__ __forceinline__ float2 swiglu32x2(float2 g, float2 u) {
    const float2 d = __fadd2_rn(make_float2(1.0f, 1.0f), exp32x2_neg(g));
    return __fmul2_rn(__fmul2_rn(g, make_float2(__frcp_rn(d.x), __frcp_rn(d.y))), u);
}

constexpr int SG_THREADS = 256;
constexpr int SG_MAXCH = 8;   // 16-byte chunks of h per thread: I <= 256 x 8 x 8
constexpr int SG_WARP_ROW_MAX_I = 32 * SG_MAXCH * 8;   // rows this short go one per warp

// WARP_ROWS: one warp per row (8 rows per CTA, no block-wide step) for I <= 2048.  With a CTA per row a short row
// leaves most threads idle and pays a CTA launch and a barrier for 3 KB of input: MoE down projection, I = 768,
// 65536 rows: the expert layer with this kernel in it took 561 us with a CTA per row and 437 us with a warp per
// row (the kernel alone: 74 us, 3.4 TB/s of the 5 bytes per element it moves).
template <bool QUANT, bool WARP_ROWS>
__global__ void __launch_bounds__(SG_THREADS, 5)
swiglu_fp8_kernel(const uint16_t* __restrict__ GU, int64_t ldg, int M, int I, uint16_t* __restrict__ Hout, int64_t ldh,
                  uint8_t* __restrict__ x8, float* __restrict__ sx) {
    __shared__ float s_red[SG_THREADS / 32];
    grid_launch_dependents();
    grid_dependency_wait();
    const int r = WARP_ROWS ? blockIdx.x * (SG_THREADS / 32) + (threadIdx.x >> 5) : blockIdx.x;
    if (WARP_ROWS && r >= M) return;   // the whole warp
    const int tid = WARP_ROWS ? (threadIdx.x & 31) : threadIdx.x;   // position inside the row's team
    constexpr int TEAM = WARP_ROWS ? 32 : SG_THREADS;
    const uint4* grow = reinterpret_cast<const uint4*>(GU + (int64_t)r * ldg);
    const uint4* urow = reinterpret_cast<const uint4*>(GU + (int64_t)r * ldg + I);
    const int nch = I / 8;

    uint4 h[SG_MAXCH];
    __nv_bfloat162 am2 = as_bf162(0u);
#pragma unroll
    for (int i = 0; i < SG_MAXCH; ++i) {
        const int c = tid + i * TEAM;
        h[i] = make_uint4(0u, 0u, 0u, 0u);
        if (c < nch) {
            const uint4 g4 = grow[c], u4 = urow[c];
            const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w}, uw[4] = {u4.x, u4.y, u4.z, u4.w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 h2 = swiglu32x2(make_float2(__uint_as_float(gw[j] << 16), __uint_as_float(gw[j] & 0xFFFF0000u)),
                                             make_float2(__uint_as_float(uw[j] << 16), __uint_as_float(uw[j] & 0xFFFF0000u)));
                o[j] = bf162_bits(__floats2bfloat162_rn(h2.x, h2.y));
            }
            h[i] = make_uint4(o[0], o[1], o[2], o[3]);
            if (QUANT) {   // packed bf16 magnitudes, two at a time
                const __nv_bfloat162 m2 = __hmax2(__hmax2(__habs2(as_bf162(o[0])), __habs2(as_bf162(o[1]))),
                                                  __hmax2(__habs2(as_bf162(o[2])), __habs2(as_bf162(o[3]))));
                am2 = __hmax2(am2, m2);
            }
            if (!QUANT) *reinterpret_cast<uint4*>(Hout + (int64_t)r * ldh + c * 8) = h[i];
        }
    }
    if (!QUANT) return;
    uint32_t am = max(bf162_bits(am2) & 0xFFFFu, bf162_bits(am2) >> 16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
    float amax = __uint_as_float(am << 16);
    if (!WARP_ROWS) {
        if ((tid & 31) == 0) s_red[tid >> 5] = amax;
        __syncthreads();
        amax = s_red[0];
#pragma unroll
        for (int i = 1; i < SG_THREADS / 32; ++i) amax = fmaxf(amax, s_red[i]);
    }
    const float amaxp = fmaxf(amax, __uint_as_float((uint32_t)(127 - 40) << 23));
    const float scale = __fdiv_rn(amaxp, 448.0f);
    const float inv = __fdiv_rn(448.0f, amaxp);
    if (tid == 0) sx[r] = scale;
    uint8_t* orow = x8 + (int64_t)r * I;
#pragma unroll
    for (int i = 0; i < SG_MAXCH; ++i) {
        const int c = tid + i * TEAM;
        if (c < nch) {
            const uint32_t w[4] = {h[i].x, h[i].y, h[i].z, h[i].w};
            uint32_t e[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 sc = __fmul2_rn(make_float2(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xFFFF0000u)),
                                             make_float2(inv, inv));
                e[j] = e4m3x2(sc.x, sc.y) & 0xFFFFu;
            }
            *reinterpret_cast<uint2*>(orow + c * 8) = make_uint2(e[0] | (e[1] << 16), e[2] | (e[3] << 16));
        }
    }
}

// quant: Hout unused; else x8 / sx unused.  I <= 16384, a multiple of 8.
template <bool QUANT>
static cudaError_t launch_swiglu_rows(const void* GU, int64_t ldg, int M, int I, void* Hout, int64_t ldh, void* x8, void* sx,
                                      cudaStream_t st) {
    if (I <= SG_WARP_ROW_MAX_I)
        return launch_pdl(swiglu_fp8_kernel<QUANT, true>, dim3((M + SG_THREADS / 32 - 1) / (SG_THREADS / 32)), dim3(SG_THREADS), 0,
                          st, static_cast<const uint16_t*>(GU), ldg, M, I, static_cast<uint16_t*>(Hout), ldh,
                          static_cast<uint8_t*>(x8), static_cast<float*>(sx));
    return launch_pdl(swiglu_fp8_kernel<QUANT, false>, dim3(M), dim3(SG_THREADS), 0, st, static_cast<const uint16_t*>(GU), ldg, M,
                      I, static_cast<uint16_t*>(Hout), ldh, static_cast<uint8_t*>(x8), static_cast<float*>(sx));
}
cudaError_t launch_swiglu_fp8(bool quant, const void* GU, int64_t ldg, int M, int I, void* Hout, int64_t ldh, void* x8,
                              void* sx, cudaStream_t st) {
    if (M <= 0) return cudaSuccess;
    return quant ? launch_swiglu_rows<true>(GU, ldg, M, I, Hout, ldh, x8, sx, st)
                 : launch_swiglu_rows<false>(GU, ldg, M, I, Hout, ldh, x8, sx, st);
}

}  // namespace osc
