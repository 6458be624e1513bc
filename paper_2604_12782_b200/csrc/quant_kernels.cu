// Memory-bound kernels of the OSC path:
//   quant_extract_kernel : Algorithm 2 fused - table lookup, back-up of the flagged channels into
//                          the dense buffer B (xo), zero-out, CalculateScale (E8M0), Quantize (E2M1),
//                          scales written straight into the 128x4 block layout the tensor core reads.
//   fp8_quant_kernel     : Section 3.4 fallback - per-row dynamic E4M3 with an fp32 scale.
//   build_sched_kernel   : grouped (MoE) tile schedule from the expert offsets.
// All three are used for activations (online) and for weights (offline preparation).
#include <cuda_bf16.h>

#include "common.cuh"

namespace osc {

// ---------------------------------------------------------------- conversions
__device__ __forceinline__ uint32_t e2m1x2(float lo, float hi) {
    uint16_t r;
    asm("{ .reg .b8 t;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\t"
        "mov.b16 %0, {t, 0}; }"
        : "=h"(r)
        : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t u) { return *reinterpret_cast<__nv_bfloat162*>(&u); }
__device__ __forceinline__ uint32_t bf162_bits(__nv_bfloat162 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// ------------------------------------------------------- Algorithm 2, fused
// Persistent kernel, two CTAs per SM.  A producer warp streams 128-row x 128-channel tiles of X
// (32 KB, as two 64-channel halves with the 128-byte swizzle) through a shared-memory ring with
// TMA.  Each of the 512 consumer threads owns one 32-channel group of one row of the tile, 64 bytes
// of shared memory that no other thread touches:
//   1. back-up + zero-out: for every flagged channel of its group (bit mask of the table) the thread
//      copies the element from the shared tile into xo (the buffer B) and overwrites it with +0;
//   2. it loads its 64 bytes, releases the slot, then amax, E8M0 code, exact fp32 scaling, hardware
//      E2M1 conversion, one 16-byte store of the packed codes; the four scale bytes of a row are
//      gathered by shuffles into one 32-bit word of the 128 x 4 scale block.
// No block-wide barrier: a version that first ran step 1 as (row, channel) tasks over all threads
// and staged the scale block in shared memory spent a large part of its time waiting at the barrier
// between the steps.
constexpr int QE_ROWS = 128;
constexpr int QE_COLS = 128;
constexpr int QE_CONSUMERS = 512;               // = groups per tile
constexpr int QE_THREADS = QE_CONSUMERS + 32;
constexpr int QE_HALF_BYTES = QE_ROWS * 128;    // 64 channels x 128 rows
constexpr int QE_TILE_BYTES = 2 * QE_HALF_BYTES;
constexpr int QE_STAGES = 3;
constexpr int QE_CTAS_PER_SM = 2;
constexpr int QE_SMEM = QE_STAGES * QE_TILE_BYTES + 1024 + 256;

// byte offset of channel `col` (0..127) of row `row` inside a swizzled tile
__device__ __forceinline__ int qe_elem_offset(int row, int col) {
    const int half = col >> 6, within = (col & 63) * 2;
    return half * QE_HALF_BYTES + row * 128 + ((((within >> 4) ^ (row & 7))) << 4) + (within & 15);
}

// eight fp32 values -> eight E2M1 codes packed into 32 bits (element 0 in the low nibble)
__device__ __forceinline__ uint32_t e2m1x8(float f0, float f1, float f2, float f3, float f4, float f5, float f6,
                                           float f7) {
    uint32_t r;
    asm("{ .reg .b8 t0, t1, t2, t3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7;\n\t"
        "mov.b32 %0, {t0, t1, t2, t3}; }"
        : "=r"(r)
        : "f"(f0), "f"(f1), "f"(f2), "f"(f3), "f"(f4), "f"(f5), "f"(f6), "f"(f7));
    return r;
}

// FMT_MXFP4: groups of 32, E8M0 scale (Algorithm 2 as the paper states it).  FMT_NVFP4: blocks of 16, unsigned
// E4M3 block scale, tensor-level scale 2^tensor_e (the G = 16 variant): t = fl32(amax' * fl32(1/6)),
// scale byte = E4M3(t), elements = E2M1(fl32(x' * fl32(1/scale))) with x' = x * 2^-tensor_e, backed-up
// channels stored as bf16(x').
constexpr int FMT_MXFP4 = 0;
constexpr int FMT_NVFP4 = 1;

// NVFP4 arithmetic of one 32-channel group held as 16 packed bf16 pairs: two blocks of 16, per block
// t = fl32(amax' * fl32(1/6)) with amax' the block maximum in the scaled domain (x * p2, p2 = 2^-tensor_e, exact),
// scale byte = E4M3(t) nearest-even saturating, codes = E2M1(fl32(x * fac)) with fac = fl32(1/scale) * p2.
// Returns the two scale bytes (block 0 in bits 7:0) and the 32 packed codes in q.
__device__ __forceinline__ uint32_t nvfp4_group(const uint32_t (&w)[16], float p2, uint32_t (&q)[4]) {
    uint32_t codes = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        __nv_bfloat162 m2 = __habs2(as_bf162(w[8 * h]));
#pragma unroll
        for (int i = 1; i < 8; ++i) m2 = __hmax2(m2, __habs2(as_bf162(w[8 * h + i])));
        const uint32_t am2 = bf162_bits(m2);
        const float amax = __uint_as_float(max(am2 & 0xFFFFu, am2 >> 16) << 16) * p2;   // exact
        const float t = __fmul_rn(amax, __fdiv_rn(1.0f, 6.0f));
        const uint32_t sb = e4m3x2(t, 0.0f) & 0xFFu;          // nearest-even, saturating at 448
        codes |= sb << (8 * h);
        // value of the scale byte: exponent field e, mantissa m -> (8 + m) * 2^(e - 10), or m * 2^-9
        const int se = (int)(sb >> 3), sm = (int)(sb & 7u);
        const float sbv = se ? __uint_as_float((uint32_t)(se + 120) << 23) * (1.0f + 0.125f * (float)sm)
                             : 0.001953125f * (float)sm;
        // one factor per block: fl32(1/scale) times the (exact) power of two of the tensor scale
        const float fac = sbv > 0.0f ? __fdiv_rn(1.0f, sbv) * p2 : 0.0f;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            float f[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t u = w[8 * h + 4 * i + j];
                f[2 * j] = __fmul_rn(__uint_as_float(u << 16), fac);
                f[2 * j + 1] = __fmul_rn(__uint_as_float(u & 0xFFFF0000u), fac);
            }
            q[2 * h + i] = e2m1x8(f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
        }
    }
    return codes;
}

// MXFP4 arithmetic of one 32-channel group held as 16 packed bf16 pairs (Algorithm 2, CalculateScale + Quantize).
// Returns the E8M0 code and the 32 packed E2M1 codes in q.
__device__ __forceinline__ int mxfp4_group(const uint32_t (&w)[16], uint32_t (&q)[4]) {
    // amax on the bf16 magnitudes, two at a time
    __nv_bfloat162 m8[8];   // a tree, not a chain of sixteen: the thread has little else to overlap it with
#pragma unroll
    for (int i = 0; i < 8; ++i) m8[i] = __hmax2(__habs2(as_bf162(w[2 * i])), __habs2(as_bf162(w[2 * i + 1])));
    const __nv_bfloat162 m2 = __hmax2(__hmax2(__hmax2(m8[0], m8[1]), __hmax2(m8[2], m8[3])),
                                      __hmax2(__hmax2(m8[4], m8[5]), __hmax2(m8[6], m8[7])));
    const uint32_t am2 = bf162_bits(m2);
    const uint32_t am = max(am2 & 0xFFFFu, am2 >> 16);
    // CalculateScale: E8M0 code = biased exponent of amax - 2, floored at 0 (2^(floor(log2 amax) - 2))
    const int ex = (int)(am >> 7);
    int code = max(ex - 2, 0);
    if (ex == 255) code = 255;
    // Quantize: x * 2^(127 - code) is exact (a power of two, two bf16 values per multiply; results below
    // the bf16 normal range are far under the 0.25 tie point and keep their sign), then hardware E2M1
    // rounding (nearest-even, saturating) of the fp32 extensions
    const __nv_bfloat162 inv2 = as_bf162(((uint32_t)(254 - min(code, 253)) << 7) * 0x10001u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float f[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t p = bf162_bits(__hmul2(as_bf162(w[4 * i + j]), inv2));
            f[2 * j] = __uint_as_float(p << 16);
            f[2 * j + 1] = __uint_as_float(p & 0xFFFF0000u);
        }
        q[i] = e2m1x8(f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
    }
    return code;
}

// bf16 bits of x * 2^-tensor_e rounded to bf16 (nearest even): the backed-up channel in the scaled domain of NVFP4
__device__ __forceinline__ uint16_t nvfp4_backup(uint16_t b, int tensor_e) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(
        __uint_as_float((uint32_t)b << 16) * __uint_as_float((uint32_t)(127 - tensor_e) << 23)));
}

template <int FMT>
__global__ void __launch_bounds__(QE_THREADS, QE_CTAS_PER_SM)
quant_extract_kernel(const __grid_constant__ CUtensorMap tm_x, int M, int K,
                     const uint32_t* __restrict__ mask, const int32_t* __restrict__ prefix,
                     const int32_t* __restrict__ idx_o,
                     uint8_t* __restrict__ xq, uint8_t* __restrict__ sf, uint16_t* __restrict__ xo,
                     int Ko, int Kop, const int32_t* __restrict__ sched, int max_tiles, int tensor_e) {
    extern __shared__ uint8_t qe_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(qe_smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + QE_STAGES * QE_TILE_BYTES);
    uint64_t* empty_bar = full_bar + QE_STAGES;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + QE_STAGES);

    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < QE_STAGES; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], QE_CONSUMERS / 32);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tm_x);
    }
    __syncthreads();
    grid_launch_dependents();
    grid_dependency_wait();   // X may come from, and the outputs may still be read by, earlier kernels

    const int ncb = K / QE_COLS;  // 128-channel blocks per row
    const int nrt = sched ? sched[0] : (M + QE_ROWS - 1) / QE_ROWS;
    const int total = nrt * ncb;
    // each CTA takes a contiguous run of tiles (channel block fastest), so neighbours in time are
    // neighbours in memory and the (row tile, channel block) pair advances without divisions
    const int per_cta = (total + gridDim.x - 1) / gridDim.x;
    const int t_begin = min(total, (int)blockIdx.x * per_cta);
    const int t_end = min(total, t_begin + per_cta);

    if (warp == QE_CONSUMERS / 32) {
        // ------------------------------------------------------------------ producer
        int s = 0;
        uint32_t ph = 0;
        int rt = t_begin / ncb, cb = t_begin - rt * ncb;
        for (int t = t_begin; t < t_end; ++t) {
            const int row0 = sched ? sched[1 + rt] : rt * QE_ROWS;
            if (!wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, 21)) break;
            if (elect_one()) {
                mbar_arrive_expect_tx(&full_bar[s], QE_TILE_BYTES);
                tma_load_2d(smem + s * QE_TILE_BYTES, &tm_x, &full_bar[s], cb * QE_COLS, row0);
                tma_load_2d(smem + s * QE_TILE_BYTES + QE_HALF_BYTES, &tm_x, &full_bar[s], cb * QE_COLS + 64, row0);
            }
            __syncwarp();
            if (++s == QE_STAGES) { s = 0; ph ^= 1u; }
            if (++cb == ncb) { cb = 0; ++rt; }
        }
    } else {
        // ----------------------------------------------------------------- consumers
        // Every thread owns one 32-channel group of one row of the tile (64 bytes of the shared tile that no
        // other thread touches), so back-up, zero-out, scale and quantization need no block-wide barrier.
        const int tid = threadIdx.x;
        const int grow = tid >> 2;  // my row inside the tile
        const int gi = tid & 3;     // my group inside the 128-channel block
        int s = 0;
        uint32_t ph = 0;
        int rt = t_begin / ncb, cb = t_begin - rt * ncb;
        // the table entries of the next tile are fetched one tile ahead, so their latency is off the critical path
        uint32_t flagged_next = 0;
        int slot_next = 0;
        if (t_begin < t_end) {
            flagged_next = mask[cb * 4 + gi];
            slot_next = prefix[cb * 4 + gi];
        }
        for (int t = t_begin; t < t_end; ++t) {
            int row0, row_end, sf_row0;
            if (sched) {
                row0 = sched[1 + rt];
                row_end = sched[1 + max_tiles + rt];
                sf_row0 = sched[1 + 2 * max_tiles + rt];
            } else {
                row0 = rt * QE_ROWS;
                row_end = M;
                sf_row0 = row0;
            }
            const int r = row0 + grow;
            uint32_t flagged = flagged_next;
            int slot = slot_next;
            if (t + 1 < t_end) {
                const int cbn = (cb + 1 == ncb) ? 0 : cb + 1;
                flagged_next = mask[cbn * 4 + gi];
                slot_next = prefix[cbn * 4 + gi];
            }
            if (!wait_bounded(&full_bar[s], ph, abort_flag, 22)) break;
            uint8_t* st = smem + s * QE_TILE_BYTES;
            const uint8_t* rowp = st + (gi >> 1) * QE_HALF_BYTES + grow * 128;

            // step 1: back-up of my group's flagged channels into xo, zero-out in the shared tile
            const bool had_flagged = flagged != 0;
            while (flagged) {
                const int j = __ffs(flagged) - 1;
                flagged &= flagged - 1;
                const int within = (((gi & 1) << 5) + j) * 2;   // byte inside the 128-byte half row
                uint16_t* e = reinterpret_cast<uint16_t*>(const_cast<uint8_t*>(rowp) +
                                                          ((((within >> 4) ^ (grow & 7))) << 4) + (within & 15));
                if (r < row_end) {
                    uint16_t b = *e;
                    if (FMT == FMT_NVFP4) b = nvfp4_backup(b, tensor_e);   // into the scaled domain of the block-scaled path
                    xo[(int64_t)r * Kop + slot] = b;
                }
                ++slot;
                *e = 0;
            }

            // step 2: my group into registers, then release the slot
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + (((((gi & 1) << 2) + i) ^ (grow & 7)) << 4));
                w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
            }
            // the zero-out above wrote the slot through the generic proxy; the next TMA load overwrites it through
            // the async proxy, so the writes are fenced before the slot is handed back
            if (had_flagged) fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);
            if (++s == QE_STAGES) { s = 0; ph ^= 1u; }

            if (FMT == FMT_MXFP4) {
            int code = 0;
            if (r < row_end) {  // rows past the end (next expert / padding) count as zeros: code 0, nothing stored
                uint32_t q[4];
                code = mxfp4_group(w, q);
                *reinterpret_cast<uint4*>(xq + (int64_t)r * (K / 2) + cb * (QE_COLS / 2) + gi * 16) =
                    make_uint4(q[0], q[1], q[2], q[3]);
            }
            // the four scale bytes of a row and 128-channel block are one 32-bit word of the block layout:
            // gather them from the four lanes of the row, lane gi == 0 stores
            uint32_t word = (uint32_t)code << (8 * gi);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
            if (gi == 0) {
                const int64_t blk = (int64_t)(sf_row0 / 128) * (K / 128) + cb;
                *reinterpret_cast<uint32_t*>(sf + blk * 512 + (grow & 31) * 16 + (grow >> 5) * 4) = word;
            }
            } else {
            // NVFP4: my 32 channels are two blocks of 16
            uint32_t codes = 0;
            if (r < row_end) {
                uint32_t q[4];
                codes = nvfp4_group(w, __uint_as_float((uint32_t)(127 - tensor_e) << 23), q);
                *reinterpret_cast<uint4*>(xq + (int64_t)r * (K / 2) + cb * (QE_COLS / 2) + gi * 16) =
                    make_uint4(q[0], q[1], q[2], q[3]);
            }
            // scale blocks cover 64 channels: lanes gi = 0,1 hold the four bytes of one word, gi = 2,3 of the next
            uint32_t word = codes << (16 * (gi & 1));
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
            if ((gi & 1) == 0) {
                const int64_t blk = (int64_t)(sf_row0 / 128) * (K / 64) + cb * 2 + (gi >> 1);
                *reinterpret_cast<uint32_t*>(sf + blk * 512 + (grow & 31) * 16 + (grow >> 5) * 4) = word;
            }
            }

            // zero the pad columns of xo once per row tile
            if (cb == 0 && Kop > Ko) {
                const int npad = Kop - Ko;
                for (int i = tid; i < QE_ROWS * npad; i += QE_CONSUMERS) {
                    const int rr = row0 + i / npad;
                    if (rr < row_end) xo[(int64_t)rr * Kop + Ko + i % npad] = 0;
                }
            }
            if (++cb == ncb) { cb = 0; ++rt; }
        }
    }
}

// ------------------------------------------------------ per-row dynamic E4M3
// One CTA per row.  The row is kept in registers between the amax pass and the encode pass
// when it fits (K <= 256 threads x 8 chunks x 8 elements = 16384), else re-read.
constexpr int F8_THREADS = 256;
constexpr int F8_MAXCH = 8;

__global__ void __launch_bounds__(F8_THREADS)
fp8_quant_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M, int K, uint8_t* __restrict__ x8,
                 float* __restrict__ sx) {
    __shared__ float s_red[F8_THREADS / 32];
    grid_launch_dependents();
    grid_dependency_wait();
    const int r = blockIdx.x;
    const uint16_t* xrow = X + (int64_t)r * ldx;
    const int nch = K / 8;  // 16-byte chunks in the row
    const int tid = threadIdx.x;

    uint4 v[F8_MAXCH];
    uint32_t am = 0;
#pragma unroll
    for (int i = 0; i < F8_MAXCH; ++i) {
        const int c = tid + i * F8_THREADS;
        if (c < nch) {
            v[i] = *reinterpret_cast<const uint4*>(xrow + c * 8);
            am = max(am, max(max(v[i].x & 0x7FFFu, (v[i].x >> 16) & 0x7FFFu), max(v[i].y & 0x7FFFu, (v[i].y >> 16) & 0x7FFFu)));
            am = max(am, max(max(v[i].z & 0x7FFFu, (v[i].z >> 16) & 0x7FFFu), max(v[i].w & 0x7FFFu, (v[i].w >> 16) & 0x7FFFu)));
        }
    }
    for (int c = tid + F8_MAXCH * F8_THREADS; c < nch; c += F8_THREADS) {
        const uint4 u = *reinterpret_cast<const uint4*>(xrow + c * 8);
        am = max(am, max(max(u.x & 0x7FFFu, (u.x >> 16) & 0x7FFFu), max(u.y & 0x7FFFu, (u.y >> 16) & 0x7FFFu)));
        am = max(am, max(max(u.z & 0x7FFFu, (u.z >> 16) & 0x7FFFu), max(u.w & 0x7FFFu, (u.w >> 16) & 0x7FFFu)));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = __uint_as_float(am << 16);
    __syncthreads();
    float amax = s_red[0];
#pragma unroll
    for (int i = 1; i < F8_THREADS / 32; ++i) amax = fmaxf(amax, s_red[i]);

    // amax' = max(amax, 2^-40); sx = amax'/448; inv = 448/amax' (IEEE fp32 divisions)
    const float amaxp = fmaxf(amax, __uint_as_float((uint32_t)(127 - 40) << 23));
    const float scale = __fdiv_rn(amaxp, 448.0f);
    const float inv = __fdiv_rn(448.0f, amaxp);
    if (tid == 0) sx[r] = scale;

    auto encode8 = [&](const uint4& u) -> uint2 {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
        uint32_t h[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __fmul_rn(__uint_as_float(w[i] << 16), inv);
            const float hi = __fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), inv);
            h[i] = e4m3x2(lo, hi) & 0xFFFFu;
        }
        return make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
    };
    uint8_t* orow = x8 + (int64_t)r * K;
#pragma unroll
    for (int i = 0; i < F8_MAXCH; ++i) {
        const int c = tid + i * F8_THREADS;
        if (c < nch) *reinterpret_cast<uint2*>(orow + c * 8) = encode8(v[i]);
    }
    for (int c = tid + F8_MAXCH * F8_THREADS; c < nch; c += F8_THREADS) {
        const uint4 u = *reinterpret_cast<const uint4*>(xrow + c * 8);
        *reinterpret_cast<uint2*>(orow + c * 8) = encode8(u);
    }
}

// Short rows (K <= 4096): one warp per row, eight rows per CTA, the row held in registers
// (at most 8 or 16 chunks of 8 elements per lane).  A CTA per row leaves most threads idle or
// spends its time in the block-wide reduction.
template <int F8W_MAXCH>
__global__ void __launch_bounds__(256)
fp8_quant_rows_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M, int K, uint8_t* __restrict__ x8,
                      float* __restrict__ sx) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (r >= M) return;
    const uint16_t* xrow = X + (int64_t)r * ldx;
    const int nch = K / 8;
    uint4 v[F8W_MAXCH];
    uint32_t am = 0;
#pragma unroll
    for (int i = 0; i < F8W_MAXCH; ++i) {
        const int c = lane + i * 32;
        if (c < nch) {
            v[i] = *reinterpret_cast<const uint4*>(xrow + c * 8);
            am = max(am, max(max(v[i].x & 0x7FFFu, (v[i].x >> 16) & 0x7FFFu), max(v[i].y & 0x7FFFu, (v[i].y >> 16) & 0x7FFFu)));
            am = max(am, max(max(v[i].z & 0x7FFFu, (v[i].z >> 16) & 0x7FFFu), max(v[i].w & 0x7FFFu, (v[i].w >> 16) & 0x7FFFu)));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
    const float amax = __uint_as_float(am << 16);
    const float amaxp = fmaxf(amax, __uint_as_float((uint32_t)(127 - 40) << 23));
    const float scale = __fdiv_rn(amaxp, 448.0f);
    const float inv = __fdiv_rn(448.0f, amaxp);
    if (lane == 0) sx[r] = scale;
    uint8_t* orow = x8 + (int64_t)r * K;
#pragma unroll
    for (int i = 0; i < F8W_MAXCH; ++i) {
        const int c = lane + i * 32;
        if (c < nch) {
            const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
            uint32_t h[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float lo = __fmul_rn(__uint_as_float(w[k] << 16), inv);
                const float hi = __fmul_rn(__uint_as_float(w[k] & 0xFFFF0000u), inv);
                h[k] = e4m3x2(lo, hi) & 0xFFFFu;
            }
            *reinterpret_cast<uint2*>(orow + c * 8) = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
        }
    }
}

// ------------------------------------------------ MXFP8 (E4M3 elements, E8M0 scale per 32)
// The 8-bit micro-scaling form of the fallback (Section 3.4).  One warp per row; per step the warp
// reads 512 contiguous bytes (256 channels, 16 bytes per lane), so four neighbouring lanes hold one
// 32-channel group: amax by two shuffles, scale code = biased exponent of amax - 8 (floored at 0),
// exact power-of-two scaling in fp32, hardware E4M3 rounding, 8 bytes stored per lane (256
// contiguous bytes per warp).  The scale bytes of four consecutive groups are one 32-bit word of the
// 128 x 4 block layout; lanes 0 and 16 gather and store them.  Rows between M and the next multiple
// of 128 only get zero scale bytes, so that the GEMM never reads an uninitialised scale block.
constexpr int MX8_ROWS_PER_CTA = 8;

__global__ void __launch_bounds__(32 * MX8_ROWS_PER_CTA)
mxfp8_quant_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M, int M_pad, int K, uint8_t* __restrict__ x8,
                   uint8_t* __restrict__ sf, const int32_t* __restrict__ sched, int max_tiles, int kspan) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    // Dense: scale row = tensor row.  Grouped: the warp index runs over the scale rows of the 128-row tile schedule
    // (every expert starts on a 128-row scale block); scale rows past an expert's end get zero bytes.
    const int v = blockIdx.x * MX8_ROWS_PER_CTA + (threadIdx.x >> 5);
    int r = v, sr = v;
    bool valid = v < M;
    if (sched) {
        const int tile = v >> 7;
        if (tile >= sched[0]) return;
        r = sched[1 + tile] + (v & 127);
        valid = r < sched[1 + max_tiles + tile];
        sr = sched[1 + 2 * max_tiles + tile] + (v & 127);
    } else if (v >= M_pad) {
        return;
    }
    const int katoms = K / 128;
    // scale word of (scale row sr, 128-channel block a): block (sr/128)*katoms + a, word (sr%32)*4 + (sr%128)/32
    uint32_t* sf_row = reinterpret_cast<uint32_t*>(sf + (size_t)(sr / 128) * katoms * 512) + (sr & 31) * 4 + ((sr & 127) >> 5);
    // blockIdx.y splits the row into spans of kspan channels (a multiple of 1024), so that few rows still fill the GPU
    const int k_begin = blockIdx.y * kspan, k_end = min(K, k_begin + kspan);
    if (!valid) {
        for (int a = k_begin / 128 + lane; a < k_end / 128; a += 32) sf_row[(size_t)a * 128] = 0u;
        return;
    }
    const uint4* xrow = reinterpret_cast<const uint4*>(X + (int64_t)r * ldx);
    uint2* orow = reinterpret_cast<uint2*>(x8 + (int64_t)r * K);
    const int nch = k_end / 8;  // 16-byte chunks up to the end of my span
    constexpr int U = 4;        // independent loads in flight per lane
    for (int c0 = k_begin / 8; c0 < nch; c0 += 32 * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * 32 + lane;
            v[u] = (c < nch) ? xrow[c] : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * 32 + lane;
            if (c0 + u * 32 >= nch) break;  // warp-uniform
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            uint32_t am = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) am = max(am, max(w[i] & 0x7FFFu, (w[i] >> 16) & 0x7FFFu));
            am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
            am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 2));
            const int ex = (int)(am >> 7);
            int code = max(ex - 8, 0);
            if (ex == 255) code = 255;
            const float inv = __uint_as_float((uint32_t)(254 - min(code, 253)) << 23);
            uint32_t h[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __uint_as_float(w[i] << 16) * inv;
                const float hi = __uint_as_float(w[i] & 0xFFFF0000u) * inv;
                h[i] = e4m3x2(lo, hi) & 0xFFFFu;
            }
            if (c < nch) orow[c] = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
            // groups 0-3 of this step live in lanes 0,4,8,12 and groups 4-7 in lanes 16,20,24,28
            const int base = lane & 16;
            const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, (uint32_t)code, base);
            const uint32_t b1 = __shfl_sync(0xFFFFFFFFu, (uint32_t)code, base + 4);
            const uint32_t b2 = __shfl_sync(0xFFFFFFFFu, (uint32_t)code, base + 8);
            const uint32_t b3 = __shfl_sync(0xFFFFFFFFu, (uint32_t)code, base + 12);
            const int a = (c0 + u * 32) / 16 + (lane >> 4);  // 128-channel block of this half-warp
            if ((lane & 15) == 0 && a < katoms) sf_row[(size_t)a * 128] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
        }
    }
}


// ------------------------------- dynamic-protection control group (Section 4.2): run-time extraction
// Per token and 32-channel group the element of largest magnitude is found at run time (ties: lowest
// channel), kept in bf16 and removed; the rest is MXFP4 as in Algorithm 2.  Same thread layout as the
// MXFP8 quantizer: one warp per row, 16 bytes (8 channels) per lane and step, four lanes per group.
// Outputs per step: 4 bytes of packed codes per lane, the dense high-precision operand xo (the
// extracted element at its own channel, +0 elsewhere: 16 bytes per lane), and per group one scale
// byte, one index byte and the bf16 value (gathered by shuffles, written by lanes 0 and 16).
__global__ void __launch_bounds__(32 * MX8_ROWS_PER_CTA)
dyn_quant_extract_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M, int M_pad, int K, uint8_t* __restrict__ xq,
                         uint8_t* __restrict__ sf, uint16_t* __restrict__ xo, uint8_t* __restrict__ idx,
                         uint16_t* __restrict__ val) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * MX8_ROWS_PER_CTA + (threadIdx.x >> 5);
    if (r >= M_pad) return;
    const int katoms = K / 128;
    const int Kg = K / 32;
    uint32_t* sf_row = reinterpret_cast<uint32_t*>(sf + (size_t)(r / 128) * katoms * 512) + (r & 31) * 4 + ((r & 127) >> 5);
    if (r >= M) {
        for (int a = lane; a < katoms; a += 32) sf_row[(size_t)a * 128] = 0u;
        return;
    }
    const uint4* xrow = reinterpret_cast<const uint4*>(X + (int64_t)r * ldx);
    uint32_t* qrow = reinterpret_cast<uint32_t*>(xq + (int64_t)r * (K / 2));
    uint4* orow = reinterpret_cast<uint4*>(xo + (int64_t)r * K);
    const int nch = K / 8;
    const int sub = lane & 3;       // my quarter of the group
    for (int c0 = 0; c0 < nch; c0 += 32) {
        const int c = c0 + lane;
        const bool live = c < nch;  // K is a multiple of 128, so a group is never split by the end of the row
        const uint4 v = live ? xrow[c] : make_uint4(0u, 0u, 0u, 0u);
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
        // key = |x| (15 bits) above (31 - local channel): the maximum picks the largest magnitude, then the lowest channel
        uint32_t key = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t a = (w[i >> 1] >> ((i & 1) * 16)) & 0x7FFFu;
            key = max(key, (a << 5) | (uint32_t)(31 - (sub * 8 + i)));
        }
        key = max(key, __shfl_xor_sync(0xFFFFFFFFu, key, 1));
        key = max(key, __shfl_xor_sync(0xFFFFFFFFu, key, 2));
        const int jstar = 31 - (int)(key & 31u);
        const bool mine = (jstar >> 3) == sub;
        const int istar = jstar & 7;
        // the extracted element: bit copy out of the owning lane, +0 in its place
        uint32_t picked = 0;
        uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (mine && (istar >> 1) == k) {
                const uint32_t keep = (istar & 1) ? 0x0000FFFFu : 0xFFFF0000u;
                picked = (istar & 1) ? (w[k] >> 16) : (w[k] & 0xFFFFu);
                o[k] = w[k] & ~keep;
                w[k] &= keep;
            }
        }
        picked = __shfl_sync(0xFFFFFFFFu, picked, (lane & ~3) + (jstar >> 3));
        if (live) orow[c] = make_uint4(o[0], o[1], o[2], o[3]);
        // CalculateScale / Quantize of what is left (as in Algorithm 2)
        uint32_t am = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) am = max(am, max(w[i] & 0x7FFFu, (w[i] >> 16) & 0x7FFFu));
        am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
        am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 2));
        const int ex = (int)(am >> 7);
        int code = max(ex - 2, 0);
        if (ex == 255) code = 255;
        const float inv = __uint_as_float((uint32_t)(254 - min(code, 253)) << 23);
        const uint32_t q = e2m1x8(__uint_as_float(w[0] << 16) * inv, __uint_as_float(w[0] & 0xFFFF0000u) * inv,
                                  __uint_as_float(w[1] << 16) * inv, __uint_as_float(w[1] & 0xFFFF0000u) * inv,
                                  __uint_as_float(w[2] << 16) * inv, __uint_as_float(w[2] & 0xFFFF0000u) * inv,
                                  __uint_as_float(w[3] << 16) * inv, __uint_as_float(w[3] & 0xFFFF0000u) * inv);
        if (live) qrow[c] = q;
        // per-group outputs: groups 0-3 of the step sit in lanes 0,4,8,12, groups 4-7 in lanes 16,20,24,28
        const int base = lane & 16;
        uint32_t sfw = 0, idw = 0, v01 = 0, v23 = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            sfw |= __shfl_sync(0xFFFFFFFFu, (uint32_t)code, base + 4 * k) << (8 * k);
            idw |= __shfl_sync(0xFFFFFFFFu, (uint32_t)jstar, base + 4 * k) << (8 * k);
            const uint32_t pv = __shfl_sync(0xFFFFFFFFu, picked, base + 4 * k);
            if (k < 2) v01 |= pv << (16 * k); else v23 |= pv << (16 * (k - 2));
        }
        const int g0 = c0 / 4 + (lane >> 4) * 4;   // first of my half-warp's four groups
        if ((lane & 15) == 0 && g0 < Kg) {
            sf_row[(size_t)(g0 / 4) * 128] = sfw;
            *reinterpret_cast<uint32_t*>(idx + (int64_t)r * Kg + g0) = idw;
            *reinterpret_cast<uint2*>(val + (int64_t)r * Kg + g0) = make_uint2(v01, v23);
        }
    }
}


// ------------------------------------------------------------ grouped schedule
// sched[0] = number of row tiles (tile_rows = 128 or 256 rows each, never crossing an expert boundary);
// then four arrays of max_tiles entries: first row, end row (exclusive, the expert's end), first scale
// row (scale rows are padded to 128 per expert whatever the tile height), expert.
// Block 0 builds the 128-row schedule (if sched is given), block 1 the 256-row one (if sched2 is given).  Thread e scans
// expert e's tile count and padded scale rows block-wide, then thread t writes tile t (binary search for its expert):
// a version with a serial prefix by one thread and one thread per expert took ~14 us for 128 experts.
constexpr int SCHED_THREADS = 1024;   // = the most experts a schedule can be built for

__global__ void __launch_bounds__(SCHED_THREADS)
build_sched_kernel(const int32_t* __restrict__ off, int E, int32_t* __restrict__ sched128, int max_tiles128,
                   int32_t* __restrict__ sched256, int max_tiles256) {
    __shared__ int s_tiles[SCHED_THREADS + 1];    // exclusive prefix of the experts' tile counts (+ the total)
    __shared__ int s_sfbase[SCHED_THREADS];       // exclusive prefix of the experts' padded scale rows
    __shared__ int s_wt[32], s_ws[32];
    grid_launch_dependents();
    grid_dependency_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool tall = blockIdx.x == 1 || sched128 == nullptr;
    int32_t* sched = tall ? sched256 : sched128;
    const int max_tiles = tall ? max_tiles256 : max_tiles128;
    const int tile_rows = tall ? 256 : 128;
    if (sched == nullptr) return;
    // thread e owns expert e: block-wide exclusive scan of (tiles, padded scale rows)
    const int m = tid < E ? off[tid + 1] - off[tid] : 0;
    const int nt = (m + tile_rows - 1) / tile_rows, ns = (m + 127) / 128 * 128;
    int it = nt, is = ns;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xFFFFFFFFu, it, o), b = __shfl_up_sync(0xFFFFFFFFu, is, o);
        if (lane >= o) { it += a; is += b; }
    }
    if (lane == 31) { s_wt[warp] = it; s_ws[warp] = is; }
    __syncthreads();
    if (warp == 0) {
        int a = s_wt[lane], b = s_ws[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xFFFFFFFFu, a, o), y = __shfl_up_sync(0xFFFFFFFFu, b, o);
            if (lane >= o) { a += x; b += y; }
        }
        s_wt[lane] = a;
        s_ws[lane] = b;
    }
    __syncthreads();
    const int base_t = warp ? s_wt[warp - 1] : 0, base_s = warp ? s_ws[warp - 1] : 0;
    s_tiles[tid] = base_t + it - nt;
    s_sfbase[tid] = base_s + is - ns;
    const int total = s_wt[31];
    if (tid == 0) {
        s_tiles[SCHED_THREADS] = total;
        sched[0] = total < max_tiles ? total : max_tiles;
    }
    __syncthreads();
    // thread t owns tile t: its expert is the last one whose first tile is <= t
    for (int t = tid; t < total && t < max_tiles; t += SCHED_THREADS) {
        int lo = 0, hi = E - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (s_tiles[mid] <= t) lo = mid; else hi = mid - 1;
        }
        const int e = lo;   // (experts without rows share their first tile index with the next one; the last of them owns it)
        const int i = t - s_tiles[e];
        sched[1 + t] = off[e] + i * tile_rows;
        sched[1 + max_tiles + t] = off[e + 1];
        sched[1 + 2 * max_tiles + t] = s_sfbase[e] + i * tile_rows;
        sched[1 + 3 * max_tiles + t] = e;
    }
}

// ----------------------------------------------- per-tile copy of weight scales
// dst holds, for every bn-row tile of the weight matrix, ceil(bn/128) 128-row scale blocks per
// 128-channel block in which the tile's first row is row 0 (rows past the tile or past N: code 0).
// Block order: [tile][block of the tile][K block]; inside a block the usual 512-byte arrangement.
// gate_up: the matrix holds gate rows [0, N/2) above up rows [N/2, N) and tile t covers bn/2 gate features followed
// by the same bn/2 up features: row j of the tile is matrix row t*bn/2 + j (j < bn/2) or N/2 + t*bn/2 + j - bn/2.
// sf_channels: channels per scale block (128: MXFP4 / MXFP8, 64: NVFP4).
__global__ void retile_sf_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int N, int K, int bn, int gate_up,
                                 int sf_channels) {
    const int katoms = K / sf_channels;
    const int atoms_per_tile = (bn + 127) / 128;
    const int ntiles = (N + bn - 1) / bn;
    const int64_t total = (int64_t)ntiles * atoms_per_tile * katoms * 512;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int byte = (int)(i & 511);
        const int64_t blk = i >> 9;
        const int ka = (int)(blk % katoms);
        const int at = (int)((blk / katoms) % atoms_per_tile);
        const int tile = (int)(blk / ((int64_t)katoms * atoms_per_tile));
        const int r32 = byte >> 4, q = (byte >> 2) & 3, g4 = byte & 3;
        const int j = at * 128 + q * 32 + r32;  // row inside the tile
        int n = tile * bn + j;
        bool valid = j < bn && n < N;
        if (gate_up) {
            const int hb = bn / 2, f = tile * hb + (j < hb ? j : j - hb);   // feature
            n = (j < hb ? 0 : N / 2) + f;
            valid = j < bn && f < N / 2;
        }
        uint8_t v = 0;
        if (valid)
            v = src[((int64_t)(n / 128) * katoms + ka) * 512 + (n % 32) * 16 + ((n % 128) / 32) * 4 + g4];
        dst[i] = v;
    }
}

cudaError_t launch_retile_sf(const uint8_t* src, uint8_t* dst, int N, int K, int bn, cudaStream_t st, bool gate_up,
                             int sf_channels) {
    const int64_t total = (int64_t)((N + bn - 1) / bn) * ((bn + 127) / 128) * (K / sf_channels) * 512;
    if (total <= 0) return cudaSuccess;
    const int blocks = (int)((total + 255) / 256 < 2048 ? (total + 255) / 256 : 2048);
    retile_sf_kernel<<<blocks, 256, 0, st>>>(src, dst, N, K, bn, gate_up ? 1 : 0, sf_channels);
    return cudaGetLastError();
}

// ------------------------------------------------------------ end of a weight preparation
// The quantizers signal their dependents at their first instruction, so with programmatic launches a
// kernel two launches further down the stream can begin (up to its own grid_dependency_wait) while a
// weight quantizer is still writing; the few-row GEMM uses exactly that freedom to stream weights ahead
// of its wait.  Weights therefore must be complete before any later launch can begin: every
// *_prepare_* call ends with this kernel, launched without the programmatic attribute (it starts after
// everything before it on the stream has finished and its writes are visible) and without an early
// trigger (whatever follows starts after it has finished).
__global__ void prepare_fence_kernel() {}

cudaError_t launch_prepare_fence(cudaStream_t st) {
    prepare_fence_kernel<<<1, 32, 0, st>>>();
    return cudaGetLastError();
}

// ------------------------------------------------- gather of quantized rows (MoE dispatch)
// In a mixture-of-experts layer every token goes to several experts, and Algorithm 2 does not depend on the expert
// (one table per layer): the tokens are quantized once, and this kernel copies each token's packed codes, scale bytes
// and backed-up channels to the rows its experts own (row_token[r] = source token of permuted row r).  One block per
// 128-row tile of the schedule, one warp per row at a time; scale bytes move as the 32-bit words of the 128 x 4 block
// layout; the scale rows that only pad an expert's last block are written as zeros.
constexpr int GQ_WARPS = 16;              // warps per block; each takes 128 / GQ_WARPS rows of the tile
constexpr int GQ_RPW = 128 / GQ_WARPS;

__global__ void __launch_bounds__(32 * GQ_WARPS)
gather_quantized_kernel(const int32_t* __restrict__ row_token, int T, int K, int Kop, int katoms,
                        const uint8_t* __restrict__ xq_u, const uint8_t* __restrict__ sf_u, const uint16_t* __restrict__ xo_u,
                        uint8_t* __restrict__ xq, uint8_t* __restrict__ sf, uint16_t* __restrict__ xo,
                        const int32_t* __restrict__ sched, int max_tiles) {
    extern __shared__ uint32_t gq_sf[];   // the tile's scale block row: [K / 128][128] words, written out in one piece
    grid_launch_dependents();
    grid_dependency_wait();
    const int tile = blockIdx.x;
    if (tile >= sched[0]) return;
    const int row0 = sched[1 + tile], row_end = sched[1 + max_tiles + tile], sf_row0 = sched[1 + 2 * max_tiles + tile];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // katoms: scale blocks along K (K / 128 for MXFP4, K / 64 for NVFP4)
    const int nq = K / 32;          // 16-byte chunks of a row of packed codes
    const int no = Kop / 8;         // 16-byte chunks of a row of backed-up channels
    const uint32_t* sfu32 = reinterpret_cast<const uint32_t*>(sf_u);
    uint32_t* sf32 = reinterpret_cast<uint32_t*>(sf);
    // the warp's rows (rr = warp, warp + GQ_WARPS, ...): lane i holds the token of row i; four rows per pass, all
    // their loads issued before the first store
    const int my_r = row0 + warp + GQ_WARPS * (lane % GQ_RPW);
    const int my_t = (my_r < row_end) ? min(max(row_token[my_r], 0), T - 1) : -1;   // an index outside the token range
                                                                                 // must not become an address
    for (int i0 = 0; i0 < GQ_RPW; i0 += 4) {
        uint4 q[4][2], o4[4];
        uint32_t sw[4];
        int tk[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            tk[u] = __shfl_sync(0xFFFFFFFFu, my_t, i0 + u);
            q[u][0] = q[u][1] = o4[u] = make_uint4(0u, 0u, 0u, 0u);
            sw[u] = 0u;
            if (tk[u] >= 0) {
                const uint4* src_q = reinterpret_cast<const uint4*>(xq_u + (size_t)tk[u] * (K / 2));
                if (lane < nq) q[u][0] = src_q[lane];
                if (lane + 32 < nq) q[u][1] = src_q[lane + 32];
                if (lane < no) o4[u] = reinterpret_cast<const uint4*>(xo_u + (size_t)tk[u] * Kop)[lane];
                if (lane < katoms)
                    sw[u] = sfu32[((size_t)(tk[u] >> 7) * katoms + lane) * 128 + (tk[u] & 31) * 4 + ((tk[u] & 127) >> 5)];
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int rr = warp + GQ_WARPS * (i0 + u);
            const int r = row0 + rr, sr = sf_row0 + rr;
            // scale words: the row's own, or zeros for the rows that only pad the expert's last scale block; staged
            // in shared memory (every tile starts a 128-row scale block, so rr is the row inside the block)
            uint32_t* dst_sf = gq_sf + (rr & 31) * 4 + (rr >> 5);
            if (lane < katoms) dst_sf[lane * 128] = sw[u];
            for (int a = lane + 32; a < katoms; a += 32)
                dst_sf[a * 128] = tk[u] >= 0 ? sfu32[((size_t)(tk[u] >> 7) * katoms + a) * 128 + (tk[u] & 31) * 4 + ((tk[u] & 127) >> 5)] : 0u;
            (void)sr;
            if (tk[u] < 0) continue;
            uint4* dst_q = reinterpret_cast<uint4*>(xq + (size_t)r * (K / 2));
            if (lane < nq) dst_q[lane] = q[u][0];
            if (lane + 32 < nq) dst_q[lane + 32] = q[u][1];
            for (int c = lane + 64; c < nq; c += 32)
                dst_q[c] = reinterpret_cast<const uint4*>(xq_u + (size_t)tk[u] * (K / 2))[c];
            uint4* dst_o = reinterpret_cast<uint4*>(xo + (size_t)r * Kop);
            if (lane < no) dst_o[lane] = o4[u];
            for (int c = lane + 32; c < no; c += 32) dst_o[c] = reinterpret_cast<const uint4*>(xo_u + (size_t)tk[u] * Kop)[c];
        }
    }
    __syncthreads();
    uint4* dst_blk = reinterpret_cast<uint4*>(sf32 + (size_t)(sf_row0 >> 7) * katoms * 128);
    for (int i = threadIdx.x; i < katoms * 32; i += blockDim.x) dst_blk[i] = reinterpret_cast<const uint4*>(gq_sf)[i];
}

cudaError_t launch_gather_quantized(const int32_t* row_token, int T, int K, int Kop, const void* xq_u, const void* sf_u,
                                    const void* xo_u, void* xq, void* sf, void* xo, const int32_t* sched, int max_tiles,
                                    cudaStream_t st, int sf_channels) {
    if (max_tiles <= 0) return cudaSuccess;
    const int katoms = K / sf_channels;
    static PerDevice configured;   // the tile's scale block row is staged in shared memory: beyond 48 KB it must be asked for
    if ((size_t)katoms * 512 > 48 * 1024)
        if (cudaError_t e = opt_in_shared_memory(configured, gather_quantized_kernel, 160 * 1024)) return e;
    return launch_pdl(gather_quantized_kernel, dim3(max_tiles), dim3(32 * GQ_WARPS), (size_t)katoms * 512, st, row_token, T, K, Kop, katoms,
                      static_cast<const uint8_t*>(xq_u), static_cast<const uint8_t*>(sf_u), static_cast<const uint16_t*>(xo_u),
                      static_cast<uint8_t*>(xq), static_cast<uint8_t*>(sf), static_cast<uint16_t*>(xo), sched, max_tiles);
}

// ------------------------------------------------------------------ launchers
template <int FMT>
static cudaError_t launch_quant_extract_fmt(const CUtensorMap& tm_x, int M, int K, const uint32_t* mask,
                                            const int32_t* prefix, const int32_t* idx_o, void* xq, void* sf, void* xo,
                                            int Ko, int Kop, const int32_t* sched, int max_tiles, int num_sms,
                                            int tensor_e, cudaStream_t st) {
    const int tiles = (sched ? max_tiles : (M + QE_ROWS - 1) / QE_ROWS) * (K / QE_COLS);
    if (tiles <= 0) return cudaSuccess;
    static PerDevice configured;
    if (cudaError_t e = opt_in_shared_memory(configured, quant_extract_kernel<FMT>, QE_SMEM)) return e;
    const int grid = tiles < QE_CTAS_PER_SM * num_sms ? tiles : QE_CTAS_PER_SM * num_sms;
    return launch_pdl(quant_extract_kernel<FMT>, dim3(grid), dim3(QE_THREADS), QE_SMEM, st, tm_x, M, K, mask, prefix,
                      idx_o, static_cast<uint8_t*>(xq), static_cast<uint8_t*>(sf), static_cast<uint16_t*>(xo), Ko, Kop,
                      sched, max_tiles, tensor_e);
}

cudaError_t launch_quant_extract(const CUtensorMap& tm_x, int M, int K, const uint32_t* mask,
                                 const int32_t* prefix, const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko, int Kop,
                                 const int32_t* sched, int max_tiles, int num_sms, cudaStream_t st) {
    return launch_quant_extract_fmt<FMT_MXFP4>(tm_x, M, K, mask, prefix, idx_o, xq, sf, xo, Ko, Kop, sched, max_tiles,
                                               num_sms, 0, st);
}
// NVFP4 / G = 16 form (dense only): tensor-level scale 2^tensor_e
cudaError_t launch_quant_extract_nvfp4(const CUtensorMap& tm_x, int M, int K, const uint32_t* mask,
                                       const int32_t* prefix, const int32_t* idx_o, void* xq, void* sf, void* xo, int Ko,
                                       int Kop, int num_sms, int tensor_e, cudaStream_t st, const int32_t* sched,
                                       int max_tiles) {
    return launch_quant_extract_fmt<FMT_NVFP4>(tm_x, M, K, mask, prefix, idx_o, xq, sf, xo, Ko, Kop, sched, max_tiles, num_sms,
                                               tensor_e, st);
}

cudaError_t launch_fp8_quant(const void* X, int64_t ldx, int M, int K, void* x8, void* sx, cudaStream_t st) {
    if (M <= 0) return cudaSuccess;
    if (K <= 8 * 32 * 8)
        return launch_pdl(fp8_quant_rows_kernel<8>, dim3((M + 7) / 8), dim3(256), 0, st, static_cast<const uint16_t*>(X),
                          ldx, M, K, static_cast<uint8_t*>(x8), static_cast<float*>(sx));
    if (K <= 16 * 32 * 8) {
        return launch_pdl(fp8_quant_rows_kernel<16>, dim3((M + 7) / 8), dim3(256), 0, st, static_cast<const uint16_t*>(X),
                          ldx, M, K, static_cast<uint8_t*>(x8), static_cast<float*>(sx));
    }
    return launch_pdl(fp8_quant_kernel, dim3(M), dim3(F8_THREADS), 0, st, static_cast<const uint16_t*>(X), ldx, M, K,
                      static_cast<uint8_t*>(x8), static_cast<float*>(sx));
}

cudaError_t launch_mxfp8_quant(const void* X, int64_t ldx, int M, int K, void* x8, void* sf, const int32_t* sched,
                               int max_tiles, cudaStream_t st) {
    if (M <= 0) return cudaSuccess;
    const int M_pad = sched ? max_tiles * 128 : (M + 127) / 128 * 128;
    // one warp per (row, span of 1024 channels = one pass of the warp's loop): few rows still fill the GPU, and
    // with many rows it costs nothing (measured the same as whole rows per warp at M = 8192)
    const int kspan = 1024;
    return launch_pdl(mxfp8_quant_kernel, dim3((M_pad + MX8_ROWS_PER_CTA - 1) / MX8_ROWS_PER_CTA, (K + kspan - 1) / kspan),
                      dim3(32 * MX8_ROWS_PER_CTA), 0, st, static_cast<const uint16_t*>(X), ldx, M, M_pad, K,
                      static_cast<uint8_t*>(x8), static_cast<uint8_t*>(sf), sched, max_tiles, kspan);
}

cudaError_t launch_dyn_quant_extract(const void* X, int64_t ldx, int M, int K, void* xq, void* sf, void* xo, void* idx,
                                     void* val, cudaStream_t st) {
    if (M <= 0) return cudaSuccess;
    const int M_pad = (M + 127) / 128 * 128;
    return launch_pdl(dyn_quant_extract_kernel, dim3((M_pad + MX8_ROWS_PER_CTA - 1) / MX8_ROWS_PER_CTA),
                      dim3(32 * MX8_ROWS_PER_CTA), 0, st, static_cast<const uint16_t*>(X), ldx, M, M_pad, K,
                      static_cast<uint8_t*>(xq), static_cast<uint8_t*>(sf), static_cast<uint16_t*>(xo),
                      static_cast<uint8_t*>(idx), static_cast<uint16_t*>(val));
}

cudaError_t launch_build_sched(const int32_t* off, int E, int32_t* sched128, int max_tiles128, int32_t* sched256,
                               int max_tiles256, cudaStream_t st) {
    const int blocks = (sched128 != nullptr) + (sched256 != nullptr);
    if (blocks == 0) return cudaSuccess;
    return launch_pdl(build_sched_kernel, dim3(blocks), dim3(SCHED_THREADS), 0, st, off, E, sched128, max_tiles128, sched256,
                      max_tiles256);
}

}  // namespace osc
