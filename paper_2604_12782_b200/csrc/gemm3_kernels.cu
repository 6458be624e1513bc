// Few-row ("decode") variant of the tensor-core kernels: up to 64 activation rows (two CTAs per SM) or up to 256
// (one CTA per SM), dense weights.
//
// With a handful of tokens the linear layer streams its weights once and is bound by HBM bandwidth and
// by latency, not by the tensor cores (the memory-bound column of the paper's efficiency table,
// M = 16-64).  The roles of the operands are swapped: a CTA owns 128 OUTPUT FEATURES (weight rows), which
// become the 128 rows of the MMA, and the tokens become its N dimension (16..256), so no tensor-core row
// is spent on padding and a stage moves 16 KB of weights for 2-8 KB of activations (up to 32 KB in the
// 256-row form).  To put every SM on the weight stream, the K loop of one 128-feature tile is split over the S CTAs of a thread-block
// cluster; each CTA accumulates its K slice in its own TMEM, parks the fp32 partial tile in its shared
// memory, and after a cluster barrier every CTA adds, in rank order, the partials of its share of the
// tokens through distributed shared memory (deterministic, no global scratch, no atomics) and writes
// those bf16 outputs.
//
// The weight tiles do not depend on the kernel that quantized the activations, so the producer issues
// its first ring of weight loads BEFORE the programmatic-dependency wait: the weight stream overlaps the
// activation quantizer.
//
//   warp 0    : TMA producer          warp 1 : MMA issuer, TMEM owner        warps 2-5 : epilogue
// QX form (MXFP4, up to 16 rows): no quantizer kernel runs in front.  The scales of Algorithm 2 are local to a
// 32-channel group, so a CTA can quantize exactly the activations of its own K slice: while the weight stream is in
// flight, warps 2-5 read the bf16 rows of X, zero the flagged channels, compute scale and codes with the
// quantizer's own arithmetic and write the stage's activation tile (128-byte swizzle), its scale blocks, and for
// the blocks of Path B the gathered flagged channels, straight into the ring.  Every cluster of a feature tile
// repeats this for the same few rows (they come from L2), which costs less than a kernel boundary.
// Modes and K-block order are those of the other GEMM kernels (Path A block-scaled FP4 blocks - MXFP4 or
// NVFP4 - then the BF16 blocks of Path B; or E4M3 blocks with per-row scales applied in the epilogue, or
// block-scaled E4M3).
#include <cuda_bf16.h>

#include "common.cuh"

namespace osc {

namespace decode {

constexpr int MODE_OSC = 0;
constexpr int MODE_FP8 = 1;
constexpr int MODE_MXF8 = 2;            // block-scaled FP8 (MXFP8): one 128-channel scale block per stage and operand
constexpr int MODE_NVF4 = 3;            // Eq. 5 on NVFP4: E4M3 scale per 16 channels (four 64-channel scale blocks per
                                        // stage), BF16 branch, power-of-two output scale
constexpr int BF = 128;                 // output features per CTA = MMA rows = TMEM lanes
constexpr int ROW_BYTES = 128;
constexpr int W_BYTES = BF * ROW_BYTES;        // 16 KB of weights per stage
constexpr int THREADS = 192;
constexpr int MAX_CLUSTER = 8;
constexpr int QX_IDX_BYTES = 4096;      // QX form: the channels of up to 1024 columns of the buffer B, in shared memory

// TOK = most activation rows per call: 64 (two CTAs per SM) or 256 (one CTA per SM; for long K loops, where a
// 128-row-tile kernel would leave most SMs without a tile)
template <int MODE, int TOK>
struct Cfg {
    static constexpr bool SCALED = MODE != MODE_FP8;
    static constexpr bool DUAL = MODE == MODE_OSC || MODE == MODE_NVF4;   // has the BF16 branch (Path B)
    static constexpr int KA = (MODE == MODE_OSC) ? 2 : (MODE == MODE_NVF4) ? 4 : 1;   // 512-byte scale blocks per stage
    static constexpr int SF_K = (MODE == MODE_NVF4) ? 64 : 128;      // channels per scale block
    static constexpr int XATOMS = (TOK > 128) ? 2 : 1;               // 128-row scale blocks of the activations
    static constexpr int X_BYTES = TOK * ROW_BYTES;                  // activations per stage
    static constexpr int SF_ROWBLOCK = (KA > 2 ? KA : 2) * 512;      // one 128-row block's scales of a stage (MXFP8 uses half)
    static constexpr int SFW_BYTES = SCALED ? SF_ROWBLOCK : 0;       // weight scales per stage
    static constexpr int SFX_BYTES = SCALED ? XATOMS * SF_ROWBLOCK : 0;   // activation scales
    static constexpr int STAGE_BYTES = W_BYTES + X_BYTES + SFW_BYTES + SFX_BYTES;
    // TOK = 64: ~105 KB per CTA, so that two CTAs share an SM (a split tile set larger than the SM count still runs in
    // one wave, and the next call's weight loads overlap this call's reduction and stores).  NVFP4's stage is 2 KB
    // larger (twice the scale bytes) and four of them miss that budget by 256 bytes: three stages there.
    static constexpr int STAGES = (MODE == MODE_NVF4 && TOK <= 64) ? 3 : 4;
    static constexpr int CTAS_PER_SM = (TOK <= 64) ? 2 : 1;
    static constexpr int TM_SFW = TOK;            // TMEM: accumulator (TOK columns), weight scales (KA blocks x 4
    static constexpr int TM_SFX = TOK + (KA > 2 ? KA : 2) * 4;   // columns), activation scales (KA x XATOMS x 4 columns)
    static_assert(TM_SFX + (KA > 2 ? KA : 2) * XATOMS * 4 <= ((TOK <= 64) ? 128 : 512), "TMEM columns");
    static constexpr int TMEM_COLS = (TOK <= 64) ? 128 : 512;
    static constexpr int PARTIAL_BYTES = TOK * BF * 4;   // parked partial tile [token][feature], aliases the first stages
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
    static_assert(STAGE_BYTES % 1024 == 0, "stage must keep 1024-byte alignment");
    static_assert(PARTIAL_BYTES <= STAGES * STAGE_BYTES, "partial tile must fit in the ring");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(cluster_addr)
                 : "memory");
    return v;
}

// QX form: NQ live row quarters of a stage (lane -> row 4j + lane/8 of quarter j, 32-channel group lane%8), quantized
// with the quantizer's arithmetic and written into the stage's activation tile (128-byte swizzle) and scale blocks.
// One straight-line body per count, so that the chains of the quarters overlap; the other quarters get zero codes
// and scales.
template <int NQ>
__device__ __forceinline__ void qx_quantize_quarters(uint32_t (&w)[4][16], uint32_t flagged, int lane, uint8_t* xt, uint8_t* sfx) {
    const int g = lane & 7;
    uint32_t q[4][4];
    int code[4];
    if (flagged) {      // zero-out: the flagged channels go through Path B
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t keep = ~(((flagged >> (2 * i)) & 1u ? 0x0000FFFFu : 0u) | ((flagged >> (2 * i + 1)) & 1u ? 0xFFFF0000u : 0u));
#pragma unroll
            for (int j = 0; j < NQ; ++j) w[j][i] &= keep;
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (j < NQ) {
            code[j] = mxfp4_group(w[j], q[j]);   // an all-zero group (row past M, channels past K): code 0, codes 0
        } else {
            code[j] = 0;
            q[j][0] = q[j][1] = q[j][2] = q[j][3] = 0u;
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int row = 4 * j + (lane >> 3);
        uint32_t word = (uint32_t)code[j] << (8 * (g & 3));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        if ((g & 3) == 0) *reinterpret_cast<uint32_t*>(sfx + (g >> 2) * 512 + (row & 31) * 16 + (row >> 5) * 4) = word;
        *reinterpret_cast<uint4*>(xt + row * ROW_BYTES + ((g ^ (row & 7)) << 4)) = make_uint4(q[j][0], q[j][1], q[j][2], q[j][3]);
    }
}

template <int MODE, int TOK, bool QX>
__global__ void __launch_bounds__(THREADS, Cfg<MODE, TOK>::CTAS_PER_SM)
gemm_decode_kernel(const __grid_constant__ GemmArgs args, const DecodeX xa) {
    using C = Cfg<MODE, TOK>;
    static_assert(!QX || (MODE == MODE_OSC && TOK <= 64), "in-kernel activation quantizer: MXFP4, few rows");
    constexpr int QWARPS = THREADS / 32 - 2;   // warps 2.. quantize in the QX form
    constexpr int STAGES = C::STAGES;
    constexpr int X_BYTES = C::X_BYTES, TM_SFW = C::TM_SFW, TM_SFX = C::TM_SFX, TMEM_COLS = C::TMEM_COLS;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * C::STAGE_BYTES);
    uint64_t* full_bar = bars;
    uint64_t* empty_bar = bars + STAGES;
    uint64_t* tfull_bar = bars + 2 * STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const int S = (int)cluster_size();
    const int rank = __shfl_sync(0xFFFFFFFFu, (int)cluster_ctarank(), 0);
    const int tile = blockIdx.x / S;
    const int n0 = tile * BF;             // first output feature of this cluster

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&full_bar[i], QX ? 2 : 1);   // the weight loads, and in the QX form the slot's quantizing warp
            mbar_init(&empty_bar[i], 1);
        }
        mbar_init(tfull_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        if (!QX) prefetch_tmap(&args.tm_a);
        prefetch_tmap(&args.tm_b);
        if (C::DUAL && args.Kop > 0) {
            if (!QX) prefetch_tmap(&args.tm_ao);
            prefetch_tmap(&args.tm_bo);
        }
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xFFFFFFFFu, *tmem_slot, 0);
    grid_launch_dependents();

    const int N = args.N, K = args.K, M = args.M;
    const int ntok = (M + 15) / 16 * 16;                       // MMA N
    const int xatoms = (ntok + 127) / 128;                     // 128-row scale blocks the activations span
    const int elems_per_kb = C::DUAL ? 256 : 128;
    const int nkb_a = (K + elems_per_kb - 1) / elems_per_kb;
    const int nkb_b = C::DUAL ? args.Kop / 64 : 0;
    const int nkb = nkb_a + nkb_b;
    const int katoms_total = K / C::SF_K;
    // my K slice: blocks [kb0, kb1) of the tile's K loop
    const int per = (nkb + S - 1) / S;
    const int kb0 = min(nkb, rank * per);
    const int kb1 = min(nkb, kb0 + per);
    const int q = warp & 3;                 // TMEM lane quarter an epilogue warp may read
    const int f = q * 32 + lane;            // my feature inside the tile
    float* partial = reinterpret_cast<float*>(smem);

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // weights (and their scales) of the first ring before the dependency wait, activations after it
        auto expect = [&](int kb, int s) {
            uint32_t bytes = W_BYTES + (QX ? 0u : (uint32_t)(ntok * ROW_BYTES));   // the activation tile holds ntok rows
            if (C::SCALED && kb < nkb_a)
                bytes += (uint32_t)(QX ? 1 : 1 + xatoms) * 512u * (uint32_t)min(C::KA, katoms_total - C::KA * kb);
            mbar_arrive_expect_tx(&full_bar[s], bytes);
        };
        auto load_w = [&](int kb, int s) {
            uint8_t* st = smem + s * C::STAGE_BYTES;
            if (kb < nkb_a) {
                tma_load_2d(st, &args.tm_b, &full_bar[s], kb * ROW_BYTES, n0);
                if (C::SCALED) {
                    const int ka = min(C::KA, katoms_total - C::KA * kb);
                    const uint8_t* sw = args.sfw + ((int64_t)tile * katoms_total + C::KA * kb) * 512;
                    bulk_load(st + W_BYTES + X_BYTES, sw, (uint32_t)ka * 512u, &full_bar[s]);
                }
            } else {
                tma_load_2d(st, &args.tm_bo, &full_bar[s], (kb - nkb_a) * 64, n0);
            }
        };
        auto load_x = [&](int kb, int s) {
            uint8_t* st = smem + s * C::STAGE_BYTES;
            if (kb < nkb_a) {
                tma_load_2d(st + W_BYTES, &args.tm_a, &full_bar[s], kb * ROW_BYTES, 0);
                if (C::SCALED) {
                    const int ka = min(C::KA, katoms_total - C::KA * kb);
                    for (int j = 0; j < xatoms; ++j)   // 128-row scale blocks of the activations
                        bulk_load(st + W_BYTES + X_BYTES + C::SFW_BYTES + j * C::SF_ROWBLOCK,
                                  args.sfa + ((int64_t)j * katoms_total + C::KA * kb) * 512, (uint32_t)ka * 512u, &full_bar[s]);
                }
            } else {
                tma_load_2d(st + W_BYTES, &args.tm_ao, &full_bar[s], (kb - nkb_a) * 64, 0);
            }
        };
        const int first = min(kb1 - kb0, STAGES);
        if (elect_one()) {
            for (int i = 0; i < first; ++i) {
                expect(kb0 + i, i);
                load_w(kb0 + i, i);
            }
        }
        __syncwarp();
        if (!QX) {
            grid_dependency_wait();   // the quantized activations come from the kernel before this one
            if (elect_one()) {
                for (int i = 0; i < first; ++i) load_x(kb0 + i, i);
            }
            __syncwarp();
        }
        int s = 0;
        uint32_t ph = 1;          // the ring has been filled once
        for (int kb = kb0 + first; kb < kb1; ++kb) {
            if (!wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, 31)) goto done;
            if (elect_one()) {
                expect(kb, s);
                load_w(kb, s);
                if (!QX) load_x(kb, s);
            }
            __syncwarp();
            if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        int s = 0;
        uint32_t ph = 0;
        const uint32_t idesc_a = (MODE == MODE_OSC)    ? idesc_mxf4(BF, ntok)
                                 : (MODE == MODE_NVF4) ? idesc_nvf4(BF, ntok)
                                 : (MODE == MODE_MXF8) ? idesc_mxf8(BF, ntok)
                                                       : idesc_e4m3(BF, ntok);
        const uint32_t idesc_b = idesc_bf16(BF, ntok);
        const uint64_t desc_hi = smem_desc_sw128(0);
        const uint64_t sf_hi = smem_desc_sf(0);
        const uint32_t smem0 = smem_u32(smem);
        for (int kb = kb0; kb < kb1; ++kb) {
            if (!wait_bounded(&full_bar[s], ph, abort_flag, 32)) goto done;
            tc_fence_after();
            const uint32_t sbase = smem0 + s * C::STAGE_BYTES;
            const uint64_t wdesc = desc_hi | (uint64_t)(sbase >> 4);               // MMA operand A: weights
            const uint64_t xdesc = desc_hi | (uint64_t)((sbase + W_BYTES) >> 4);   // MMA operand B: activations
            const uint32_t first = (kb == kb0) ? 0u : 1u;
            if (elect_one()) {
                if (MODE == MODE_OSC && kb < nkb_a) {
                    const int ka = min(2, katoms_total - 2 * kb);
                    const uint64_t sfw_d = sf_hi | (uint64_t)((sbase + W_BYTES + X_BYTES) >> 4);
                    const uint64_t sfx_d = sf_hi | (uint64_t)((sbase + W_BYTES + X_BYTES + C::SFW_BYTES) >> 4);
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        if (a < ka) {
                            tc_copy_sf(tmem_base + TM_SFW + a * 4, sfw_d + (uint64_t)(a * 32));
#pragma unroll
                            for (int j = 0; j < C::XATOMS; ++j)
                                if (j < xatoms)
                                    tc_copy_sf(tmem_base + TM_SFX + a * (C::XATOMS * 4) + j * 4, sfx_d + (uint64_t)(j * 64 + a * 32));
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (k < 2 * ka) {
                            constexpr uint32_t SFID[2] = {idesc_sf_ids(0, 0), idesc_sf_ids(2, 2)};
                            mma_mxf4(tmem_base, wdesc + 2 * k, xdesc + 2 * k, idesc_a | SFID[k & 1],
                                     tmem_base + TM_SFW + (k >> 1) * 4, tmem_base + TM_SFX + (k >> 1) * (C::XATOMS * 4),
                                     (first | (uint32_t)k) ? 1u : 0u);
                        }
                    }
                } else if (MODE == MODE_NVF4 && kb < nkb_a) {
                    // four 64-channel scale blocks per stage, one per K = 64 instruction (a whole scale column each)
                    const int ka = min(4, katoms_total - 4 * kb);
                    const uint64_t sfw_d = sf_hi | (uint64_t)((sbase + W_BYTES + X_BYTES) >> 4);
                    const uint64_t sfx_d = sf_hi | (uint64_t)((sbase + W_BYTES + X_BYTES + C::SFW_BYTES) >> 4);
#pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        if (a < ka) {
                            tc_copy_sf(tmem_base + TM_SFW + a * 4, sfw_d + (uint64_t)(a * 32));
#pragma unroll
                            for (int j = 0; j < C::XATOMS; ++j)
                                if (j < xatoms)
                                    tc_copy_sf(tmem_base + TM_SFX + a * (C::XATOMS * 4) + j * 4,
                                               sfx_d + (uint64_t)(j * (C::SF_ROWBLOCK / 16) + a * 32));
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (k < ka)
                            mma_nvf4(tmem_base, wdesc + 2 * k, xdesc + 2 * k, idesc_a, tmem_base + TM_SFW + k * 4,
                                     tmem_base + TM_SFX + k * (C::XATOMS * 4), (first | (uint32_t)k) ? 1u : 0u);
                } else if (MODE == MODE_MXF8) {
                    const uint64_t sfw_d = sf_hi | (uint64_t)((sbase + W_BYTES + X_BYTES) >> 4);
                    const uint64_t sfx_d = sf_hi | (uint64_t)((sbase + W_BYTES + X_BYTES + C::SFW_BYTES) >> 4);
                    tc_copy_sf(tmem_base + TM_SFW, sfw_d);
#pragma unroll
                    for (int j = 0; j < C::XATOMS; ++j)
                        if (j < xatoms) tc_copy_sf(tmem_base + TM_SFX + j * 4, sfx_d + (uint64_t)(j * 64));
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mma_mxf8(tmem_base, wdesc + 2 * k, xdesc + 2 * k, idesc_a | idesc_sf_ids(k, k), tmem_base + TM_SFW,
                                 tmem_base + TM_SFX, (first | (uint32_t)k) ? 1u : 0u);
                } else if (C::DUAL) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mma_f16(tmem_base, wdesc + 2 * k, xdesc + 2 * k, idesc_b, (first | (uint32_t)k) ? 1u : 0u);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mma_f8(tmem_base, wdesc + 2 * k, xdesc + 2 * k, idesc_a, (first | (uint32_t)k) ? 1u : 0u);
                }
                tc_commit(&empty_bar[s]);
            }
            __syncwarp();
            if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (elect_one()) tc_commit(tfull_bar);
        __syncwarp();
    } else if (QX) {
        // ------------------------------------------------ activations of my K slice, quantized in place (QX form)
        // Sixteen token rows at most.  Quantizing one group is a long dependent chain, so the stages are dealt to
        // the warps in turn (warp j fills ring slot j: the slots are as many as the warps) and several stages are
        // in the making at once; a lane holds (row, 32-channel group) of four row quarters for a block of Path A,
        // (row, eight flagged channels) for a block of Path B, all loads of a stage in flight before the first use.
        static_assert(!QX || STAGES == QWARPS, "one ring slot per quantizing warp");
        const int wq = warp - 2;
        const int g = lane & 7;
        int32_t* idx_s = reinterpret_cast<int32_t*>(smem + STAGES * C::STAGE_BYTES + 256);   // behind the barriers
        for (int o = (int)threadIdx.x - 64; o < args.Kop; o += QWARPS * 32) idx_s[o] = o < xa.Ko ? __ldg(xa.idx_o + o) : -1;
        asm volatile("bar.sync 1, %0;" ::"n"(QWARPS * 32) : "memory");
        grid_dependency_wait();             // X comes from the kernel before this one
        uint8_t* xt = smem + wq * C::STAGE_BYTES + W_BYTES;
        uint64_t* my_full = &full_bar[wq];
        uint32_t ph = 0;
        for (int kb = kb0 + wq; kb < kb1; kb += QWARPS) {
            uint32_t w[4][16];
            uint32_t flagged = 0u;
            const bool path_a = kb < nkb_a;
            const bool in_k = path_a && kb * 256 + g * 32 < K;
            if (in_k) flagged = __ldg(xa.mask + kb * 8 + g);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int row = 4 * j + (lane >> 3);
#pragma unroll
                for (int i = 0; i < 16; ++i) w[j][i] = 0u;
                if (row < M) {
                    const uint16_t* xrow = xa.X + (int64_t)row * xa.ldx;
                    if (in_k) {
                        const uint4* src = reinterpret_cast<const uint4*>(xrow + kb * 256 + g * 32);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint4 v = src[i];
                            w[j][4 * i] = v.x; w[j][4 * i + 1] = v.y; w[j][4 * i + 2] = v.z; w[j][4 * i + 3] = v.w;
                        }
                    } else if (!path_a) {
                        const int o0 = (kb - nkb_a) * 64 + 8 * g;
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int ch = idx_s[o0 + e];
                            if (ch >= 0) w[j][e] = xrow[ch];
                        }
                    }
                }
            }
            if (kb - kb0 >= STAGES) {       // my slot's previous stage has been multiplied
                if (!wait_bounded(&empty_bar[wq], ph, abort_flag, 34)) break;
                ph ^= 1u;
            }
            uint8_t* sfx = xt + X_BYTES + C::SFW_BYTES;
            switch (path_a ? (min(M, 16) + 3) >> 2 : 0) {   // live row quarters: straight-line code for each count
                case 1: qx_quantize_quarters<1>(w, flagged, lane, xt, sfx); break;
                case 2: qx_quantize_quarters<2>(w, flagged, lane, xt, sfx); break;
                case 3: qx_quantize_quarters<3>(w, flagged, lane, xt, sfx); break;
                case 4: qx_quantize_quarters<4>(w, flagged, lane, xt, sfx); break;
                default:                                    // a block of Path B: the gathered channels as they are
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int row = 4 * j + (lane >> 3);
                        *reinterpret_cast<uint4*>(xt + row * ROW_BYTES + ((g ^ (row & 7)) << 4)) =
                            make_uint4(w[j][0] | (w[j][1] << 16), w[j][2] | (w[j][3] << 16), w[j][4] | (w[j][5] << 16),
                                       w[j][6] | (w[j][7] << 16));
                    }
            }
            fence_proxy_async_smem();       // written through the generic proxy, read by the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(my_full);
        }
    }

done:
    // ------------------------------------------------------------------ reduction + epilogue
    // Every CTA of the cluster parks its partial tile as fp32 [token][feature] in its own shared memory (the ring
    // is free once the accumulator is complete).  After a cluster barrier CTA r sums, in rank order, the tokens
    // r, r+S, ... of all partials through distributed shared memory - a warp reads one token's 128 features as
    // one contiguous 512-byte row per peer - and stores four features per lane (8 bytes, 256 per warp and token).
    // (With the tile parked as [feature][token] every lane of a remote load hit a different row: the reduction
    // of a 256-token tile took ~15 us.)
    if (warp >= 2) {
        bool have = kb1 > kb0;
        if (have && !wait_bounded(tfull_bar, 0, abort_flag, 33)) have = false;
        tc_fence_after();
        grid_dependency_wait();             // Y may still be read by an earlier kernel
        const int n = n0 + f;
        float swn = 1.0f;
        if (MODE == MODE_FP8 && n < N) swn = args.sw[n];
        // sixteen tokens at a time: TMEM -> registers -> the parked partial tile (S > 1) or straight to Y (S == 1)
        for (int c = 0; c * 16 < ntok; ++c) {
            uint32_t r[32];   // the load fills r[0..15]
            if (have) {
                tmem_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 16), r);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) r[i] = 0u;
            }
            if (S > 1) {
#pragma unroll
                for (int i = 0; i < 16; ++i) partial[(c * 16 + i) * BF + f] = __uint_as_float(r[i]);
            } else if (n < N) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int t = c * 16 + i;
                    if (t < M) {
                        float v = __uint_as_float(r[i]);
                        if (MODE == MODE_FP8) v = v * (args.sx[t] * swn);
                        if (MODE == MODE_NVF4) v *= args.out_scale;   // back out of the scaled domain: an exact power of two
                        args.Y[(int64_t)t * args.ldy + n] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
                    }
                }
            }
        }
        tc_fence_before();
    }
    __syncwarp();
    __syncthreads();
    if (S > 1) cluster_sync_all();          // partial tiles visible to the whole cluster
    if (warp >= 2 && S > 1) {
        const int wq = warp - 2;
        const int n4 = n0 + 4 * lane;           // my four features
        float4 sw4 = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
        if (MODE == MODE_FP8 && n4 < N) sw4 = *reinterpret_cast<const float4*>(args.sw + n4);
        const uint32_t mine = smem_u32(partial) + (uint32_t)(lane * 16);
        uint32_t peer[MAX_CLUSTER];
#pragma unroll
        for (int r = 0; r < MAX_CLUSTER; ++r) peer[r] = map_to_cta(mine, (uint32_t)min(r, S - 1));
        // tokens rank, rank + S, ...; the four warps take them in turn, four tokens per pass and four peers at a
        // time (in rank order), so that up to sixteen remote loads per lane are in flight together
        for (int j = wq; rank + S * j < M; j += 16) {
            float4 v[4];
#pragma unroll
            for (int r0 = 0; r0 < MAX_CLUSTER; r0 += 4) {
                if (r0 < S) {
                    float4 p[4][4];
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const int t = rank + S * (j + 4 * h);
#pragma unroll
                        for (int r = 0; r < 4; ++r)
                            if (r0 + r < S && t < M) p[h][r] = ld_cluster_f32x4(peer[r0 + r] + (uint32_t)(t * (BF * 4)));
                    }
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            if (r0 + r < S) {
                                if (r0 + r == 0) v[h] = p[h][r];
                                else { v[h].x += p[h][r].x; v[h].y += p[h][r].y; v[h].z += p[h][r].z; v[h].w += p[h][r].w; }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int t = rank + S * (j + 4 * h);
                if (t >= M) break;
                float4 o = v[h];
                if (MODE == MODE_FP8) {
                    const float sxt = args.sx[t];
                    o.x *= sxt * sw4.x; o.y *= sxt * sw4.y; o.z *= sxt * sw4.z; o.w *= sxt * sw4.w;
                }
                if (MODE == MODE_NVF4) { o.x *= args.out_scale; o.y *= args.out_scale; o.z *= args.out_scale; o.w *= args.out_scale; }
                if (n4 < N) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
                    *reinterpret_cast<uint2*>(args.Y + (int64_t)t * args.ldy + n4) =
                        make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
                }
            }
        }
    }
    __syncwarp();
    if (S > 1) cluster_sync_all();          // nobody leaves while a peer may still read its shared memory
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag && lane == 0) atomicCAS(&g_dev_status, 0, (39 << 8) | 1);
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int MODE, int TOK, bool QX = false>
static cudaError_t launch_cfg(const GemmArgs& a, int S, cudaStream_t st, const DecodeX& xa = DecodeX{}) {
    using C = Cfg<MODE, TOK>;
    static PerDevice configured;
    constexpr int SMEM = C::SMEM_BYTES + (QX ? QX_IDX_BYTES : 0);
    if (cudaError_t e = opt_in_shared_memory(configured, gemm_decode_kernel<MODE, TOK, QX>, SMEM)) return e;
    const int tiles = (a.N + BF - 1) / BF;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles * S);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_decode_kernel<MODE, TOK, QX>, a, xa);
}

}  // namespace decode

// Cluster size (K split) of the few-row kernel: 4, 2 or 1, the largest with at most ~1.3 CTAs per SM.
// Measured on B200 (rows = 16, K = 4096): a CTA alone on its SM streams its weights at ~107 GB/s and two CTAs on
// one SM share that rate, so filling every second slot of every SM buys nothing (96 feature tiles: 9.2 us unsplit,
// 9.6 us split in 2, 14.4 us split in 3 or 4); with 48 tiles (the QKV projection) the whole linear takes 10.0 us
// with S = 4, 10.1 with S = 3, 10.9 with S = 2 or 1; with more tiles than SMs a split only adds reduction work and
// a second wave (192 tiles: 15.1 / 18.1 / 23.1 us for S = 1 / 2 / 3).  Every rank gets at least one K block.
// OSC_DECODE_SPLIT overrides.
int gemm_decode_split(int N, int nkb, int num_sms) {
    static const int forced = [] { const char* e = getenv("OSC_DECODE_SPLIT"); return e ? atoi(e) : 0; }();
    const int tiles = (N + decode::BF - 1) / decode::BF;
    int S = 1;
    if (forced > 0) S = forced;
    else if (40 * tiles <= 13 * num_sms) S = 4;
    else if (20 * tiles <= 13 * num_sms) S = 2;
    if (S > decode::MAX_CLUSTER) S = decode::MAX_CLUSTER;
    while (S > 1 && (S - 1) * ((nkb + S - 1) / S) >= nkb) --S;   // no rank without a K block
    return S;
}

cudaError_t launch_gemm_dual_decode(const GemmArgs& a, int S, cudaStream_t st) {
    return a.M <= 64 ? decode::launch_cfg<decode::MODE_OSC, 64>(a, S, st) : decode::launch_cfg<decode::MODE_OSC, 256>(a, S, st);
}
cudaError_t launch_gemm_dual_decode_quant(const GemmArgs& a, const DecodeX& xa, int S, cudaStream_t st) {
    return decode::launch_cfg<decode::MODE_OSC, 64, true>(a, S, st, xa);
}
cudaError_t launch_gemm_nvf4_decode(const GemmArgs& a, int S, cudaStream_t st) {
    return a.M <= 64 ? decode::launch_cfg<decode::MODE_NVF4, 64>(a, S, st) : decode::launch_cfg<decode::MODE_NVF4, 256>(a, S, st);
}
cudaError_t launch_gemm_mxf8_decode(const GemmArgs& a, int S, cudaStream_t st) {
    return a.M <= 64 ? decode::launch_cfg<decode::MODE_MXF8, 64>(a, S, st) : decode::launch_cfg<decode::MODE_MXF8, 256>(a, S, st);
}
cudaError_t launch_gemm_fp8_decode(const GemmArgs& a, int S, cudaStream_t st) {
    return a.M <= 64 ? decode::launch_cfg<decode::MODE_FP8, 64>(a, S, st) : decode::launch_cfg<decode::MODE_FP8, 256>(a, S, st);
}

}  // namespace osc
