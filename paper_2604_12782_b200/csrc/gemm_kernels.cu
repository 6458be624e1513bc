// Single-CTA tensor-core kernels (tcgen05 + TMEM + TMA), one persistent CTA per SM, warp-specialised.
// Used for grouped (MoE) problems and for dense problems with few rows; dense problems with many rows
// go to the CTA-pair kernel.
//   warp 0    : TMA producer (operand tiles + scale-factor blocks into a shared-memory ring)
//   warp 1    : MMA issuer (one elected lane of the converged warp) and TMEM owner
//   warps 2-9 : epilogue (TMEM -> registers -> bf16 -> swizzled shared-memory tile -> row-masked,
//               line-wide global stores)
//
// MODE_OSC : Eq. 5.  For every 128 x BN output tile the K loop first runs the block-scaled FP4
//            blocks of Path A (256 channels = 128 bytes per row and stage, four K=64 MMAs with
//            E8M0 scale vectors copied into TMEM), then the BF16 blocks of Path B over the
//            gathered channels (64 channels = 128 bytes per row and stage, four K=16 MMAs) into the
//            same fp32 accumulator.  Every stage carries 128 bytes per operand row, whatever the
//            operand type, so one ring serves both paths.
// MODE_FP8 : Section 3.4 fallback.  E4M3 x E4M3 (128 channels per stage, four K=32 MMAs); the
//            per-row activation scale and per-output-row weight scale are applied in the epilogue.
//
// MODE_MXF8: the same fallback in its 8-bit micro-scaling form: E4M3 elements with one E8M0 scale per 32
//            (128 channels and one 128-channel scale block per operand row block and stage, four K=32
//            block-scaled MMAs taking scale byte k of the TMEM column); nothing to apply in the epilogue.
// MODE_NVF4: Eq. 5 on NVFP4 (dense only): as MODE_OSC with an E4M3 scale per 16 channels - four 64-channel scale
//            blocks per stage, one whole TMEM scale column per K=64 MMA - and a power-of-two output scale in the
//            epilogue; tiles up to 192 columns wide.
//
// A tile's first row, last valid row, first scale row and expert come either from arithmetic
// (dense) or from the device-built schedule (grouped): rows past an expert's end are computed
// (they read the next expert's rows or zero fill) but never stored.
#include <cuda_bf16.h>

#include "common.cuh"

namespace osc {

constexpr int MODE_OSC = 0;
constexpr int MODE_FP8 = 1;
constexpr int MODE_MXF8 = 2;
constexpr int MODE_NVF4 = 3;   // Eq. 5 on NVFP4: E4M3 scale per 16 channels (four 64-channel scale blocks per stage), BF16
                               // branch, power-of-two output scale

constexpr int BM = 128;            // rows per tile = TMEM lanes
constexpr int ROW_BYTES = 128;     // bytes per operand row and stage (one 128-byte swizzle row)
constexpr int A_BYTES = BM * ROW_BYTES;
constexpr int G_EPI_WARPS = 8;     // two per TMEM lane quarter, each draining every other 64-column slice
constexpr int GEMM_THREADS = 64 + 32 * G_EPI_WARPS;
constexpr int TMEM_COLS = 512;
constexpr int BAND = 8;            // row tiles per scheduling band (L2 reuse of the weight tiles)
constexpr int G_EPI_TILE_BYTES = 32 * 128;  // staging tile: 32 rows x 64 bf16 columns

template <int MODE, int BN>
struct Cfg {
    static constexpr int SFB_ATOMS = (BN > 128) ? 2 : 1;  // 128-row scale blocks a tile can touch
    static constexpr bool SCALED = MODE != MODE_FP8;
    static constexpr bool DUAL = MODE == MODE_OSC || MODE == MODE_NVF4;   // has the BF16 branch (Path B)
    static constexpr int KA = (MODE == MODE_OSC) ? 2 : (MODE == MODE_NVF4) ? 4 : 1;   // 512-byte scale blocks per stage
    static constexpr int SF_K = (MODE == MODE_NVF4) ? 64 : 128;                       // channels per scale block
    static constexpr int KA_ROOM = KA > 2 ? KA : 2;
    // TMEM columns of one stage's scales (A: 4 per block, B: 4 per block and 128-row atom; MXFP8 uses half of
    // them); the FP8 mode keeps no scales in TMEM
    static constexpr int SF_COLS = SCALED ? KA_ROOM * 4 + KA_ROOM * SFB_ATOMS * 4 : 0;
    static constexpr int ACC_STAGES = (2 * BN + SF_COLS <= TMEM_COLS) ? 2 : 1;
    static constexpr int B_BYTES = BN * ROW_BYTES;
    static constexpr int SF_ROWBLOCK = KA_ROOM * 512;                // one 128-row block's scales of a stage (MXFP8 fills half)
    static constexpr int SFA_BYTES = SCALED ? SF_ROWBLOCK : 0;
    static constexpr int SFB_BYTES = SCALED ? SFB_ATOMS * SF_ROWBLOCK : 0;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;  // multiple of 1024
    static constexpr int EPI_WARP_BYTES = (BN / 64) * G_EPI_TILE_BYTES;            // one lane quarter's 32 x BN outputs
    static constexpr int EPI_BYTES = 4 * EPI_WARP_BYTES;
    static constexpr int STAGES = (224 * 1024 - EPI_BYTES) / STAGE_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
    static constexpr int TM_SFA = ACC_STAGES * BN;  // TMEM column of the activation scales
    static constexpr int TM_SFB = TM_SFA + KA_ROOM * 4;   // weight scales
    static_assert(STAGE_BYTES % 1024 == 0, "stage must keep 1024-byte alignment");
    static_assert(TM_SFA + SF_COLS <= TMEM_COLS, "TMEM budget");
    static_assert(STAGES >= 3, "ring too shallow");
    static_assert(BN % 64 == 0, "tile width");
};

struct TileInfo {
    int row0, row_end, sf_row0, expert, n0;
};

__device__ __forceinline__ int num_row_tiles(const GemmArgs& a) {
    return a.sched ? a.sched[0] : (a.M + BM - 1) / BM;
}

template <int BN>
__device__ __forceinline__ TileInfo tile_info(const GemmArgs& a, int t, int num_m, int num_n) {
    const int per_band = BAND * num_n;
    const int band = t / per_band;
    const int rem = t - band * per_band;
    const int m0 = band * BAND;
    const int h = min(BAND, num_m - m0);
    const int m = m0 + rem % h;
    const int n = rem / h;
    TileInfo ti;
    ti.n0 = n * BN;
    if (a.sched) {
        ti.row0 = a.sched[1 + m];
        ti.row_end = a.sched[1 + a.max_tiles + m];
        ti.sf_row0 = a.sched[1 + 2 * a.max_tiles + m];
        ti.expert = a.sched[1 + 3 * a.max_tiles + m];
    } else {
        ti.row0 = m * BM;
        ti.row_end = a.M;
        ti.sf_row0 = ti.row0;
        ti.expert = 0;
    }
    return ti;
}

template <int MODE, int BN>
__global__ void __launch_bounds__(GEMM_THREADS, 1) gemm_kernel(const __grid_constant__ GemmArgs args) {
    using C = Cfg<MODE, BN>;
    constexpr int STAGES = C::STAGES;
    constexpr int ACC = C::ACC_STAGES;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // [operand ring][epilogue staging tiles, 1024-byte aligned for the swizzle][barriers]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * C::STAGE_BYTES + C::EPI_BYTES);
    uint64_t* full_bar = bars;
    uint64_t* empty_bar = bars + STAGES;
    uint64_t* tfull_bar = bars + 2 * STAGES;
    uint64_t* tempty_bar = bars + 2 * STAGES + ACC;
    uint64_t* drain_bar = bars + 2 * STAGES + 2 * ACC;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2 * ACC + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    // warp-uniform values go through a shuffle so that the address arithmetic of the TMA / tcgen05
    // instructions stays in uniform registers (they are issued by one elected lane of a converged warp)
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        for (int i = 0; i < ACC; ++i) {
            mbar_init(&tfull_bar[i], 1);
            mbar_init(&tempty_bar[i], G_EPI_WARPS);
        }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&args.tm_a);
        prefetch_tmap(&args.tm_b);
        if (C::DUAL && args.Kop > 0) {
            prefetch_tmap(&args.tm_ao);
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

    const int N = args.N, K = args.K;
    const int num_n = (N + BN - 1) / BN;
    // K blocks: Path A / FP8 first, then Path B
    const int elems_per_kb = C::DUAL ? 256 : 128;
    const int nkb_a = (K + elems_per_kb - 1) / elems_per_kb;
    const int nkb_b = C::DUAL ? args.Kop / 64 : 0;
    const int nkb = nkb_a + nkb_b;
    const int katoms_total = K / C::SF_K;   // scale blocks along K
    const int natoms = (N + 127) / 128;  // 128-row scale blocks of one expert's weights
    constexpr int KA = C::KA;

    // One stage of the ring in two parts: the weight side (prepared once, never written by a kernel of the calling
    // sequence) and the activation side (the quantizer's output).  `expect` arms the stage's barrier with the bytes of both.
    auto load_weights = [&](int s, int kb, const TileInfo& ti, bool expect) {
        uint8_t* st = smem + s * C::STAGE_BYTES;
        const int brow = ti.expert * N + ti.n0;
        if (kb < nkb_a) {
            const uint32_t sfb = C::SCALED ? (uint32_t)min(KA, katoms_total - KA * kb) * 512u : 0u;   // scale bytes per row block
            if (expect) mbar_arrive_expect_tx(&full_bar[s], A_BYTES + C::B_BYTES + sfb * (1 + C::SFB_ATOMS));
            tma_load_2d(st + A_BYTES, &args.tm_b, &full_bar[s], kb * ROW_BYTES, brow);
            if (C::SCALED) {
#pragma unroll
                for (int j = 0; j < C::SFB_ATOMS; ++j) {
                    const int atom = min(ti.n0 / 128 + j, natoms - 1);
                    const uint8_t* sw = args.sfw + (((int64_t)ti.expert * natoms + atom) * katoms_total + KA * kb) * 512;
                    bulk_load(st + A_BYTES + C::B_BYTES + C::SFA_BYTES + j * C::SF_ROWBLOCK, sw, sfb, &full_bar[s]);
                }
            }
        } else {
            if (expect) mbar_arrive_expect_tx(&full_bar[s], A_BYTES + C::B_BYTES);
            tma_load_2d(st + A_BYTES, &args.tm_bo, &full_bar[s], (kb - nkb_a) * 64, brow);
        }
    };
    auto load_activations = [&](int s, int kb, const TileInfo& ti) {
        uint8_t* st = smem + s * C::STAGE_BYTES;
        if (kb < nkb_a) {
            tma_load_2d(st, &args.tm_a, &full_bar[s], kb * ROW_BYTES, ti.row0);
            if (C::SCALED) {
                const uint32_t sfb = (uint32_t)min(KA, katoms_total - KA * kb) * 512u;
                const uint8_t* sa = args.sfa + ((int64_t)(ti.sf_row0 / 128) * katoms_total + KA * kb) * 512;
                bulk_load(st + A_BYTES + C::B_BYTES, sa, sfb, &full_bar[s]);
            }
        } else {
            tma_load_2d(st, &args.tm_ao, &full_bar[s], (kb - nkb_a) * 64, ti.row0);
        }
    };

    // Dense problems: the weight side of the first tile's first ring of stages goes out BEFORE the dependency wait (the
    // CTA is resident while the quantizer in front still runs, and the weights do not depend on it); a grouped problem
    // reads its tiles from the schedule that the kernel in front builds, so nothing is known before the wait.
    const int num_m_dense = (args.M + BM - 1) / BM;
    const int pre = (args.sched == nullptr && warp == 0 && (int)blockIdx.x < num_m_dense * num_n) ? min(STAGES, nkb) : 0;
    if (pre > 0) {
        const TileInfo ti = tile_info<BN>(args, blockIdx.x, num_m_dense, num_n);
        if (elect_one()) {
            for (int kb = 0; kb < pre; ++kb) load_weights(kb, kb, ti, true);
        }
        __syncwarp();
    }
    grid_dependency_wait();   // activations (and the grouped schedule) come from the kernels before this one

    const int num_m = num_row_tiles(args);
    const int total = num_m * num_n;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        int s = 0;
        uint32_t ph = 0;
        if (pre > 0) {   // the activation side of the stages whose weight side is already under way
            const TileInfo ti = tile_info<BN>(args, blockIdx.x, num_m, num_n);
            if (elect_one()) {
                for (int kb = 0; kb < pre; ++kb) load_activations(kb, kb, ti);
            }
            __syncwarp();
            if (pre == STAGES) ph = 1u; else s = pre;
        }
        for (int t = blockIdx.x; t < total; t += gridDim.x) {
            const TileInfo ti = tile_info<BN>(args, t, num_m, num_n);
            for (int kb = (t == (int)blockIdx.x ? pre : 0); kb < nkb; ++kb) {
                if (!wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, 1)) goto done;
                if (elect_one()) {
                    load_weights(s, kb, ti, true);
                    load_activations(s, kb, ti);
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        int s = 0;
        uint32_t ph = 0;
        int acc = 0;
        uint32_t acc_ph = 0;
        constexpr uint32_t IDESC_A = (MODE == MODE_OSC)    ? idesc_mxf4(BM, BN)
                                     : (MODE == MODE_NVF4) ? idesc_nvf4(BM, BN)
                                     : (MODE == MODE_MXF8) ? idesc_mxf8(BM, BN)
                                                           : idesc_e4m3(BM, BN);
        constexpr uint32_t IDESC_B = idesc_bf16(BM, BN);
        const uint64_t desc_hi = smem_desc_sw128(0);  // everything but the start address
        const uint64_t sf_hi = smem_desc_sf(0);
        const uint32_t smem0 = smem_u32(smem);
        for (int t = blockIdx.x; t < total; t += gridDim.x) {
            const TileInfo ti = tile_info<BN>(args, t, num_m, num_n);
            if (!wait_bounded(&tempty_bar[acc], acc_ph ^ 1u, abort_flag, 2)) goto done;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
            const uint32_t sfb_tm = tmem_base + C::TM_SFB + (uint32_t)((ti.n0 % 128) / 32);
            for (int kb = 0; kb < nkb; ++kb) {
                if (!wait_bounded(&full_bar[s], ph, abort_flag, 3)) goto done;
                const uint32_t sbase = smem0 + s * C::STAGE_BYTES;
                const uint64_t adesc = desc_hi | (uint64_t)(sbase >> 4);
                const uint64_t bdesc = desc_hi | (uint64_t)((sbase + A_BYTES) >> 4);
                if (elect_one()) {
                    if (MODE == MODE_OSC && kb < nkb_a) {
                        const int ka = min(2, katoms_total - 2 * kb);
                        const uint64_t sfa_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES) >> 4);
                        const uint64_t sfb_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES + C::SFA_BYTES) >> 4);
#pragma unroll
                        for (int a = 0; a < 2; ++a) {
                            if (a < ka) {
                                tc_copy_sf(tmem_base + C::TM_SFA + a * 4, sfa_d + (uint64_t)(a * 32));
#pragma unroll
                                for (int j = 0; j < C::SFB_ATOMS; ++j)
                                    tc_copy_sf(tmem_base + C::TM_SFB + a * (C::SFB_ATOMS * 4) + j * 4,
                                               sfb_d + (uint64_t)(j * 64 + a * 32));
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if (k < 2 * ka) {
                                // byte pair inside the 4-byte scale column: 0 for the first, 2 for the second K=64 half
                                constexpr uint32_t SFID[2] = {idesc_sf_ids(0, 0), idesc_sf_ids(2, 2)};
                                mma_mxf4(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A | SFID[k & 1],
                                         tmem_base + C::TM_SFA + (k >> 1) * 4, sfb_tm + (k >> 1) * (C::SFB_ATOMS * 4),
                                         (kb | k) ? 1u : 0u);
                            }
                        }
                    } else if (MODE == MODE_NVF4 && kb < nkb_a) {
                        // four 64-channel scale blocks per stage, one per K = 64 instruction (a whole scale column each)
                        const int ka = min(4, katoms_total - 4 * kb);
                        const uint64_t sfa_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES) >> 4);
                        const uint64_t sfb_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES + C::SFA_BYTES) >> 4);
#pragma unroll
                        for (int a = 0; a < 4; ++a) {
                            if (a < ka) {
                                tc_copy_sf(tmem_base + C::TM_SFA + a * 4, sfa_d + (uint64_t)(a * 32));
#pragma unroll
                                for (int j = 0; j < C::SFB_ATOMS; ++j)
                                    tc_copy_sf(tmem_base + C::TM_SFB + a * (C::SFB_ATOMS * 4) + j * 4,
                                               sfb_d + (uint64_t)(j * (C::SF_ROWBLOCK / 16) + a * 32));
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (k < ka)
                                mma_nvf4(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A, tmem_base + C::TM_SFA + k * 4,
                                         sfb_tm + k * (C::SFB_ATOMS * 4), (kb | k) ? 1u : 0u);
                    } else if (C::DUAL) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) mma_f16(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_B, 1u);
                    } else if (MODE == MODE_MXF8) {
                        // one 128-channel scale block per stage: four K = 32 instructions, scale byte k of the column
                        const uint64_t sfa_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES) >> 4);
                        const uint64_t sfb_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES + C::SFA_BYTES) >> 4);
                        tc_copy_sf(tmem_base + C::TM_SFA, sfa_d);
#pragma unroll
                        for (int j = 0; j < C::SFB_ATOMS; ++j)
                            tc_copy_sf(tmem_base + C::TM_SFB + j * 4, sfb_d + (uint64_t)(j * 64));
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_mxf8(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A | idesc_sf_ids(k, k), tmem_base + C::TM_SFA,
                                     sfb_tm, (kb | k) ? 1u : 0u);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_f8(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A, (kb | k) ? 1u : 0u);
                    }
                    tc_commit(&empty_bar[s]);
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (elect_one()) tc_commit(&tfull_bar[acc]);
            __syncwarp();
            if (++acc == ACC) { acc = 0; acc_ph ^= 1u; }
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        // Two warps per TMEM lane quarter (32 rows); each drains every other 64-column slice into a
        // swizzled staging tile, hands the accumulator back, then writes the tile out with stores that
        // cover whole 128-byte lines (8 lanes per row, 4 rows per instruction), skipping rows past the
        // tile's last valid row.
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        int acc = 0;
        uint32_t acc_ph = 0;
        uint8_t* stage_buf = smem + STAGES * C::STAGE_BYTES + q * C::EPI_WARP_BYTES;
        for (int t = blockIdx.x; t < total; t += gridDim.x) {
            const TileInfo ti = tile_info<BN>(args, t, num_m, num_n);
            const int wrow0 = ti.row0 + q * 32;
            // FP8 scales, fetched before the wait so that their latency hides behind the K loop: the row's
            // activation scale, and per slice one coalesced load of the 64 weight scales (lane l holds
            // columns 2l, 2l+1; the conversion loop below broadcasts them with shuffles)
            float sxr = 1.0f;
            float2 wsc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            if (MODE == MODE_FP8) {
                if (wrow0 + lane < ti.row_end) sxr = args.sx[wrow0 + lane];
                const float* swp = args.sw + (int64_t)ti.expert * N;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int col = ti.n0 + (half + u * (G_EPI_WARPS / 4)) * 64 + 2 * lane;
                    if (half + u * (G_EPI_WARPS / 4) < BN / 64 && col + 1 < N)
                        wsc[u] = *reinterpret_cast<const float2*>(swp + col);
                }
            }
            if (!wait_bounded(&tfull_bar[acc], acc_ph, abort_flag, 4)) goto done;
            tc_fence_after();
            int ord = 0;
#pragma unroll 1
            for (int c = half; c < BN / 64; c += G_EPI_WARPS / 4, ++ord) {
                const float2 wv = ord == 0 ? wsc[0] : wsc[1];
                uint32_t r0[32], r1[32];
                const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c * 64);
                tmem_ld_32x32(tcol, r0);
                tmem_ld_32x32(tcol + 32, r1);
                tmem_ld_wait();
                const int col = ti.n0 + c * 64;
                uint8_t* buf = stage_buf + c * G_EPI_TILE_BYTES;
                if (col < N) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {  // 8 chunks of 16 bytes = 8 columns each
                        uint32_t o[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int cc = j * 8 + 2 * i;  // column inside the 64-column slice
                            float lo = __uint_as_float(cc < 32 ? r0[cc] : r1[cc - 32]);
                            float hi = __uint_as_float(cc < 32 ? r0[cc + 1] : r1[cc - 31]);
                            if (MODE == MODE_FP8) {
                                const float wx = __shfl_sync(0xFFFFFFFFu, wv.x, j * 4 + i);
                                const float wy = __shfl_sync(0xFFFFFFFFu, wv.y, j * 4 + i);
                                lo = lo * (sxr * wx);
                                hi = hi * (sxr * wy);
                            }
                            if (MODE == MODE_NVF4) {   // back out of the scaled domain: an exact power of two
                                lo *= args.out_scale;
                                hi *= args.out_scale;
                            }
                            const __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                            o[i] = *reinterpret_cast<const uint32_t*>(&b2);
                        }
                        // 16-byte chunk j of row `lane` lives at chunk j ^ (lane % 8): conflict-free both ways
                        *reinterpret_cast<uint4*>(buf + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                            make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
            // accumulator drained: hand it back before the stores
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty_bar[acc]);
#pragma unroll 1
            for (int c = half; c < BN / 64; c += G_EPI_WARPS / 4) {
                const int col = ti.n0 + c * 64;
                if (col >= N) break;
                const uint8_t* buf = stage_buf + c * G_EPI_TILE_BYTES;
                const int j = lane & 7;  // 16-byte chunk of the row
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    const int rl = rr * 4 + (lane >> 3);  // row inside the warp's 32
                    const int row = wrow0 + rl;
                    const uint4 v = *reinterpret_cast<const uint4*>(buf + rl * 128 + ((j ^ (rl & 7)) << 4));
                    if (row < ti.row_end) *reinterpret_cast<uint4*>(args.Y + (int64_t)row * args.ldy + col + j * 8) = v;
                }
            }
            __syncwarp();
            if (++acc == ACC) { acc = 0; acc_ph ^= 1u; }
        }
    }

done:
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag && lane == 0) {
            // gave up somewhere: let outstanding tensor-core work retire before TMEM goes away
            tc_commit(drain_bar);
            int dummy = 0;
            volatile int* never = &dummy;
            wait_bounded(drain_bar, 0, never, 5);
        }
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------- launchers
// Tile width of the single-CTA kernel: the one with the smallest (waves of tiles) x (time per K stage).  A stage
// is bound by the SM's ingest of its operands (16 KB of activations + BN x 128 bytes of weights at ~107 GB/s),
// measured on B200 at 96 stages: ~230 ns for 64 columns, ~265 ns for 128, ~390 ns for 192; 256 extrapolated.  With many
// tiles the widest wins (least time per column), with few a narrower one that still fits in one wave.
// cost_ns (optional) receives the estimate for one K stage times the waves.  OSC_BLOCK_N overrides.
int gemm_block_n(int row_tiles, int N, int num_sms, long* cost_ns, int widest) {
    static const int forced = [] {
        const char* e = getenv("OSC_BLOCK_N");
        const int v = e ? atoi(e) : 0;
        return (v == 64 || v == 128 || v == 192 || v == 256) ? v : 0;
    }();
    if (cost_ns) *cost_ns = 0;
    if (forced) return forced < widest ? forced : widest;
    const int cand[4] = {256, 192, 128, 64};
    const long stage_ns[4] = {470, 390, 265, 230};
    long best = -1;
    int best_bn = 64;
    for (int i = 0; i < 4; ++i) {
        if (cand[i] > widest) continue;
        const long tiles = (long)row_tiles * ((N + cand[i] - 1) / cand[i]);
        const long waves = (tiles + num_sms - 1) / num_sms;
        const long cost = waves * stage_ns[i];
        if (best < 0 || cost < best) { best = cost; best_bn = cand[i]; }
    }
    if (cost_ns) *cost_ns = best;
    return best_bn;
}

template <int MODE, int BN>
static cudaError_t launch_cfg(const GemmArgs& a, cudaStream_t st) {
    using C = Cfg<MODE, BN>;
    static PerDevice configured;
    if (cudaError_t e = opt_in_shared_memory(configured, gemm_kernel<MODE, BN>, C::SMEM_BYTES)) return e;
    int grid = a.num_sms;
    if (!a.sched) {
        const int total = ((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
        if (total <= 0) return cudaSuccess;
        if (total < grid) grid = total;
    }
    return launch_pdl(gemm_kernel<MODE, BN>, dim3(grid), dim3(GEMM_THREADS), C::SMEM_BYTES, st, a);
}

cudaError_t launch_gemm_dual(const GemmArgs& a, int bn, cudaStream_t st) {
    switch (bn) {
        case 64: return launch_cfg<MODE_OSC, 64>(a, st);
        case 128: return launch_cfg<MODE_OSC, 128>(a, st);
        case 192: return launch_cfg<MODE_OSC, 192>(a, st);
        default: return launch_cfg<MODE_OSC, 256>(a, st);
    }
}
cudaError_t launch_gemm_fp8(const GemmArgs& a, int bn, cudaStream_t st) {
    switch (bn) {
        case 64: return launch_cfg<MODE_FP8, 64>(a, st);
        case 128: return launch_cfg<MODE_FP8, 128>(a, st);
        case 192: return launch_cfg<MODE_FP8, 192>(a, st);
        default: return launch_cfg<MODE_FP8, 256>(a, st);
    }
}
// NVFP4: up to 192 columns (a 256-wide tile's stage, with twice the scale bytes, leaves room for two stages only)
cudaError_t launch_gemm_nvf4(const GemmArgs& a, int bn, cudaStream_t st) {
    switch (bn) {
        case 64: return launch_cfg<MODE_NVF4, 64>(a, st);
        case 128: return launch_cfg<MODE_NVF4, 128>(a, st);
        default: return launch_cfg<MODE_NVF4, 192>(a, st);
    }
}
cudaError_t launch_gemm_mxf8(const GemmArgs& a, int bn, cudaStream_t st) {
    switch (bn) {
        case 64: return launch_cfg<MODE_MXF8, 64>(a, st);
        case 128: return launch_cfg<MODE_MXF8, 128>(a, st);
        case 192: return launch_cfg<MODE_MXF8, 192>(a, st);
        default: return launch_cfg<MODE_MXF8, 256>(a, st);
    }
}

}  // namespace osc
