// CTA-pair variant of the tensor-core kernels for problems with many rows: dense, or grouped (MoE) with a
// schedule of 256-row tiles that never cross an expert boundary (rows past the expert's end are computed
// but not written).
//
// Two CTAs of a cluster (two SMs) compute one 256 x BN output tile with `cta_group::2` MMAs:
// each CTA holds 128 rows of the activation tile and its 128 x BN slice of the fp32 accumulator in
// its own TMEM, and loads only HALF of the weight tile (BN/2 rows); the tensor cores of the pair
// exchange the halves.  Per stage a CTA therefore pulls 16 KB + BN/2 x 128 B from L2 instead of
// 16 KB + BN x 128 B, which is what bounds the single-CTA kernel (L2 -> shared-memory feed).
// No cluster-multicast loads are used: every CTA fetches its own operands.
//
// Roles per CTA: warp 0 is the TMA producer, warp 1 the MMA issuer (active only in the leader CTA, rank 0;
// it also owns TMEM), then eight epilogue warps.  One elected lane of the converged issuer warp issues all
// tcgen05 instructions of a tile.  (A second producer / issuer pair working on every other tile, each on half
// of the ring, was measured and brought nothing: the tensor pipe is the limit, not the issue rate.)  Barriers:
//   full[s]   leader's only: one arrive.expect_tx by the leader's producer for the bytes of BOTH
//             CTAs; the peer's loads credit the leader's barrier (cta_group::2 loads).
//   empty[s]  one per CTA, released for both CTAs by one multicast tcgen05.commit of the leader.
//   tfull[a]  one per CTA (multicast commit); tempty[a] leader's only, one arrival per epilogue warp
//             of both CTAs (the peer's arrive through the cluster window).
// Stage layout and K-loop order are those of the single-CTA kernel (Path A FP4 blocks, then Path B
// BF16 blocks, 128 bytes per operand row and stage).
#include <cuda_bf16.h>
#include <stdio.h>

#include "common.cuh"

namespace osc {

namespace pair {

constexpr int MODE_OSC = 0;
constexpr int MODE_FP8 = 1;
constexpr int MODE_MXF8 = 2;   // block-scaled FP8 (MXFP8): scales as in MODE_OSC, no BF16 branch
constexpr int MODE_NVF4 = 3;   // Eq. 5 on NVFP4: E2M1 with an E4M3 scale per 16 channels, BF16 branch, output scale
constexpr int BM = 128;        // rows per CTA; the pair covers 256
constexpr int ROW_BYTES = 128;
constexpr int A_BYTES = BM * ROW_BYTES;
constexpr int EPI_WARPS = 8;     // two per TMEM lane quarter, each draining every other 64-column slice
constexpr int TMEM_COLS = 512;
constexpr int EPI_TILE_BYTES = 32 * 128;            // staging tile: 32 rows x 64 bf16 columns

template <int MODE, int BN>
struct Cfg {
    // Weight scales in TMEM: a tile whose first row is not a multiple of 64 would start at an odd or
    // fractional 32-row scale column (an odd column offset raised "misaligned address" on the
    // block-scaled MMA).  Such widths (240) read a per-tile copy of the weight scales, laid out at
    // weight-preparation time so that every tile starts at column 0 of its own two 128-row blocks.
    static constexpr bool TILED_SF = (BN % 64) != 0;
    // 128-row scale blocks a BN-wide tile can touch
    static constexpr int SFB_ATOMS = TILED_SF ? (BN + 127) / 128 : ((BN % 128 == 0) ? BN / 128 : BN / 128 + 1);
    static constexpr bool SCALED = MODE != MODE_FP8;
    // 128-channel scale blocks per stage and operand row block: a stage is 128 bytes per row = 256 FP4 or 128 FP8 channels
    // (NVFP4 scale blocks cover 64 channels: four per stage)
    static constexpr int KA = (MODE == MODE_OSC) ? 2 : (MODE == MODE_NVF4) ? 4 : 1;
    static constexpr bool DUAL = MODE == MODE_OSC || MODE == MODE_NVF4;   // has the BF16 branch (Path B)
    static constexpr int SF_K = (MODE == MODE_NVF4) ? 64 : 128;           // channels per scale block
    // Scale blocks of a stage that sit in TMEM at a time.  NVFP4 on 240-wide tiles has room for two of its four: the
    // issuer copies two, issues their two instructions, copies the other two into the same columns and issues theirs
    // (copies and multiplications of one thread run in the order they were issued).
    static constexpr int KA_T = (MODE == MODE_NVF4 && TILED_SF) ? 2 : KA;
    static constexpr int SF_COLS = SCALED ? KA_T * (4 + SFB_ATOMS * 4) : 0;  // TMEM columns of the scales in TMEM at a time
    static constexpr int ACC_STAGES = (2 * BN + SF_COLS <= TMEM_COLS) ? 2 : 1;
    static constexpr int SF_BUFS = (ACC_STAGES * BN + 2 * SF_COLS <= TMEM_COLS) ? 2 : 1;
    static constexpr int B_BYTES = (BN / 2) * ROW_BYTES;
    static constexpr int SFA_BYTES = SCALED ? KA * 512 : 0;
    static constexpr int SFB_BYTES = SCALED ? SFB_ATOMS * KA * 512 : 0;
    static constexpr int STAGE_BYTES = (A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES + 1023) / 1024 * 1024;
    static constexpr int THREADS = 32 * (2 + EPI_WARPS);   // producer, issuer, epilogue warps
    static constexpr int EPI_FIRST_WARP = 2;
    static constexpr int SLICES = (BN + 63) / 64;        // 64-column output slices of a tile
    static constexpr int LAST_W = BN - 64 * (SLICES - 1);  // width of the last one (64 or 48)
    // The ring's depth decides how well the operand feed rides out latency (240-wide tiles: 4 / 5 / 6 stages =
    // 112.6 / 109.5 / 106.6 us per QKV step), so the staging tiles give way to it: where staging 16 rows at a time
    // (two stores per slice) instead of 32 buys another stage, it is done.
    static constexpr int SMEM_BUDGET = 227 * 1024 - 1024 /*alignment slack*/ - 256 /*barriers*/;
    static constexpr int EPI_FULL = EPI_WARPS * EPI_TILE_BYTES;   // one 32 x 64 staging tile per epilogue warp
    static constexpr int EPI_HALVES = ((SMEM_BUDGET - EPI_FULL / 2) / STAGE_BYTES > (SMEM_BUDGET - EPI_FULL) / STAGE_BYTES) ? 2 : 1;
    static constexpr int EPI_BYTES = EPI_FULL / EPI_HALVES;
    static constexpr int STAGES = (SMEM_BUDGET - EPI_BYTES) / STAGE_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + EPI_BYTES;
    // TMEM columns.  Accumulators start at multiples of ACC_STRIDE; a 240-wide tile keeps its second
    // accumulator at column 256 and tucks the scales into the gaps (activation scales at 240..247,
    // weight scales at 496..511).
    static constexpr int ACC_STRIDE = TILED_SF ? 256 : BN;
    static constexpr int TM_SFA = TILED_SF ? BN : ACC_STAGES * BN;
    static constexpr int TM_SFB = TILED_SF ? 256 + BN : TM_SFA + 4 * KA_T;
    static constexpr int TM_SF_STRIDE = SF_COLS;         // columns of one scale buffer (when there are two)
    static constexpr uint32_t TX_A = 2u * (A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES);  // both CTAs, Path A
    static constexpr uint32_t TX_B = 2u * (A_BYTES + B_BYTES);                          // both CTAs, Path B / FP8
    static_assert(STAGE_BYTES % 1024 == 0, "stage must keep 1024-byte alignment");
    static_assert(B_BYTES % 1024 == 0, "weight half-tile must keep 1024-byte alignment");
    static_assert(TILED_SF ? (TM_SFA + 4 * KA_T <= 256 && TM_SFB + KA_T * SFB_ATOMS * 4 <= TMEM_COLS && SF_BUFS == 1)
                           : (TM_SFA + SF_BUFS * SF_COLS <= TMEM_COLS), "TMEM budget");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(STAGES >= 3, "ring too shallow");
    static_assert((SLICES + 1) / 2 <= 2, "an epilogue warp drains at most two slices of a tile");
    static_assert(BN % 16 == 0 && BN <= 256 && (LAST_W == 64 || LAST_W == 48), "tile width");
};

// GU (gate|up projection with the SwiGLU in the epilogue, MODE_OSC with per-tile weight scales, dense or grouped): the
// weight matrix holds the gate rows [0, N/2) above the up rows [N/2, N).  A tile takes BN/2 gate features and the
// same BN/2 up features - the leader CTA loads the gate half of the weight tile, its peer the up half, and the
// per-tile copy of the weight scales is arranged the same way - so accumulator columns [0, BN/2) and [BN/2, BN)
// hold gate and up of the same features, and the epilogue writes h = silu(gate) * up, BN/2 columns of
// H [M, N/2], instead of BN columns of Y.  Both are rounded to bf16 first and combined by the arithmetic of
// osc_swiglu, so H equals that call on this kernel's own Y bit for bit.
// The activation costs ~37 instructions per element, and an epilogue of eight warps (two per scheduler) runs them
// latency-bound, slower than the tile's K loop: the gate|up form has sixteen epilogue warps, one per 32-feature chunk
// and TMEM lane quarter, each with a staging tile of 16 rows x 64 bytes (two store passes per chunk).
// (Sixteen epilogue warps for the plain forms too were measured: 2-4 us slower per call on every shape - the epilogue
// there is short, and the extra warps cost registers (96 instead of 150 per thread, spills) and staging passes.)
__host__ __device__ constexpr int epi_warps(bool gu) { return gu ? 16 : EPI_WARPS; }
__host__ __device__ constexpr int pair_threads(bool gu) { return 32 * (2 + epi_warps(gu)); }

template <int MODE, int BN, bool GU = false>
__global__ void __launch_bounds__(pair_threads(GU), 1) gemm_pair_kernel(const __grid_constant__ GemmArgs args) {
    using C = Cfg<MODE, BN>;
    constexpr int EW = epi_warps(GU);
    static_assert(!GU || (MODE == MODE_OSC && C::TILED_SF && (BN / 2) % 8 == 0 && BN / 2 <= 128 &&
                          C::EPI_BYTES >= EW * 16 * 64), "gate|up epilogue: tile geometry");
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
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2 * ACC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    // warp-uniform values are passed through a shuffle so that the compiler keeps them (and all
    // address arithmetic derived from them) in uniform registers: the TMA / tcgen05 instructions
    // below are issued by one elected lane of a converged warp, not from a divergent branch
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const uint32_t rank = __shfl_sync(0xFFFFFFFFu, cluster_ctarank(), 0);  // 0 = leader
    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        for (int i = 0; i < ACC; ++i) {
            mbar_init(&tfull_bar[i], 1);
            mbar_init(&tempty_bar[i], 2 * EW);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&args.tm_a);
        prefetch_tmap(&args.tm_b);
        prefetch_tmap(&args.tm_y);
        if (C::SCALED) {
            prefetch_tmap(&args.tm_sfa);
            prefetch_tmap(&args.tm_sfw);
            if (C::DUAL && args.Kop > 0) {
                prefetch_tmap(&args.tm_ao);
                prefetch_tmap(&args.tm_bo);
            }
        }
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xFFFFFFFFu, *tmem_slot, 0);
    grid_launch_dependents();

    const int N = args.N, K = args.K;
    const int32_t* __restrict__ sched = args.sched2;
    const int elems_per_kb = C::DUAL ? 256 : 128;  // channels in 128 bytes of an operand row
    const int nkb_a = (K + elems_per_kb - 1) / elems_per_kb;
    const int nkb_b = C::DUAL ? args.Kop / 64 : 0;
    const int nkb = nkb_a + nkb_b;
    const int katoms_total = K / C::SF_K;   // scale blocks along K
    const int natoms = (N + 127) / 128;
    const int num_n = (N + BN - 1) / BN;

    // One stage of the operand ring, in two parts: the weight side (weight tile and weight scales: prepared
    // once, never written by a kernel of the calling sequence) and the activation side (this call's quantizer
    // output).  `expect` arms the leader's full barrier with the bytes of both parts and both CTAs.
    auto load_weights = [&](int s, int kb, int n0, int expert, bool expect) {
        const uint32_t st = smem_u32(smem + s * C::STAGE_BYTES);
        const uint32_t fb = map_to_cta(smem_u32(full_bar), 0) + (uint32_t)s * 8u;
        // my half of the weight rows (gate|up: the leader's half are gate rows, the peer's the up rows of the same features)
        const int brow = GU ? expert * N + (int)rank * (N / 2) + (n0 / BN) * (BN / 2) : expert * N + n0 + (int)rank * (BN / 2);
        if (kb < nkb_a) {
            if (expect && rank == 0) mbar_arrive_expect_tx(&full_bar[s], C::SCALED ? C::TX_A : C::TX_B);
            tma_load_2d_pair(st + A_BYTES, &args.tm_b, fb, kb * ROW_BYTES, brow);
            if (C::SCALED) {
#pragma unroll
                for (int j = 0; j < C::SFB_ATOMS; ++j) {
                    const int atom = C::TILED_SF ? (expert * num_n + n0 / BN) * C::SFB_ATOMS + j
                                                 : expert * natoms + min(n0 / 128 + j, natoms - 1);
                    tma_load_2d_pair(st + A_BYTES + C::B_BYTES + C::SFA_BYTES + j * (C::KA * 512), &args.tm_sfw,
                                     fb, 0, atom * katoms_total + C::KA * kb);
                }
            }
        } else {
            if (expect && rank == 0) mbar_arrive_expect_tx(&full_bar[s], C::TX_B);
            tma_load_2d_pair(st + A_BYTES, &args.tm_bo, fb, (kb - nkb_a) * 64, brow);
        }
    };
    auto load_activations = [&](int s, int kb, int row0, int sf_row0) {
        const uint32_t st = smem_u32(smem + s * C::STAGE_BYTES);
        const uint32_t fb = map_to_cta(smem_u32(full_bar), 0) + (uint32_t)s * 8u;
        const int arow = row0 + (int)rank * BM;                              // my 128 activation rows
        if (kb < nkb_a) {
            tma_load_2d_pair(st, &args.tm_a, fb, kb * ROW_BYTES, arow);
            if (C::SCALED)   // scale blocks: KA consecutive 512-byte blocks (128 channels each) per 128 rows
                tma_load_2d_pair(st + A_BYTES + C::B_BYTES, &args.tm_sfa, fb, 0,
                                 (sf_row0 / 128 + (int)rank) * katoms_total + C::KA * kb);
        } else {
            tma_load_2d_pair(st, &args.tm_ao, fb, (kb - nkb_a) * 64, arow);
        }
    };

    // Dense problems: the producer fills the ring with the weight side of its first tile BEFORE the dependency
    // wait - the CTAs of this kernel become resident while the last CTAs of the quantizer in front of it are
    // still running, and the weights do not depend on it - and adds the activation side behind the wait.
    // (Grouped problems read their tile list from a schedule that the kernel in front builds: nothing is
    // known before the wait.)
    const int num_m_dense = (args.M + 2 * BM - 1) / (2 * BM);
    const int pre = (sched == nullptr && warp == 0 && (int)blockIdx.x / 2 < num_m_dense * num_n) ? min(STAGES, nkb) : 0;
    int pre_n0 = 0, pre_row0 = 0;
    if (pre > 0) {
        const int t = blockIdx.x >> 1;
        const int per_band = args.band * num_n;
        const int band = t / per_band, rem = t - band * per_band;
        const int m0 = band * args.band, h = min(args.band, num_m_dense - m0);
        pre_n0 = (rem / h) * BN;
        pre_row0 = (m0 + rem % h) * (2 * BM);
        if (elect_one()) {
            for (int kb = 0; kb < pre; ++kb) load_weights(kb, kb, pre_n0, 0, true);
        }
        __syncwarp();
    }
    grid_dependency_wait();   // activations (and a grouped schedule) come from the kernel before this one

    const int num_m = sched ? sched[0] : num_m_dense;
    const int total = num_m * num_n;

    // tile t -> first row, column, and (grouped) last valid row, first scale row, expert
    struct Tile { int row0, n0, row_end, sf_row0, expert; };
    auto tile_of = [&](int t) {
        const int per_band = args.band * num_n;
        const int band = t / per_band;
        const int rem = t - band * per_band;
        const int m0 = band * args.band;
        const int h = min(args.band, num_m - m0);
        const int m = m0 + rem % h;
        Tile ti;
        ti.n0 = (rem / h) * BN;
        if (sched) {
            ti.row0 = sched[1 + m];
            ti.row_end = sched[1 + args.max_tiles2 + m];
            ti.sf_row0 = sched[1 + 2 * args.max_tiles2 + m];
            ti.expert = sched[1 + 3 * args.max_tiles2 + m];
        } else {
            ti.row0 = m * (2 * BM);
            ti.row_end = args.M;
            ti.sf_row0 = ti.row0;
            ti.expert = 0;
        }
        return ti;
    };

    if (warp == 0) {
        // ------------------------------------------------------- TMA producer (both CTAs)
        int s = 0;
        uint32_t ph = 0;
        if (pre > 0) {   // the activation side of the stages whose weight side is already under way
            if (elect_one()) {
                for (int kb = 0; kb < pre; ++kb) load_activations(kb, kb, pre_row0, pre_row0);
            }
            __syncwarp();
            if (pre == STAGES) ph = 1u; else s = pre;
        }
        for (int t = pair_id; t < total; t += num_pairs) {
            const Tile ti = tile_of(t);
            for (int kb = (t == pair_id ? pre : 0); kb < nkb; ++kb) {
                if (!wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, 11)) goto done;
                if (elect_one()) {
                    load_weights(s, kb, ti.n0, ti.expert, true);
                    load_activations(s, kb, ti.row0, ti.sf_row0);
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------ MMA issuer (leader CTA only, one elected lane)
        if (rank == 0) {
            int s = 0;
            uint32_t ph = 0;
            uint32_t acc_ph = 0;
            int acc = 0;
            constexpr uint32_t IDESC_A = (MODE == MODE_OSC)    ? idesc_mxf4(2 * BM, BN)
                                         : (MODE == MODE_NVF4) ? idesc_nvf4(2 * BM, BN)
                                         : (MODE == MODE_MXF8) ? idesc_mxf8(2 * BM, BN)
                                                               : idesc_e4m3(2 * BM, BN);
            constexpr uint32_t IDESC_B = idesc_bf16(2 * BM, BN);
            const uint64_t desc_hi = smem_desc_sw128(0);  // everything but the start address
            const uint64_t sf_hi = smem_desc_sf(0);
            const uint32_t ring0 = smem_u32(smem);
            for (int t = pair_id; t < total; t += num_pairs) {
                const int n0 = tile_of(t).n0;
                if (!wait_bounded(&tempty_bar[acc], acc_ph ^ 1u, abort_flag, 12)) goto done;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * C::ACC_STRIDE);
                const uint32_t sfb_tm = tmem_base + C::TM_SFB + (C::TILED_SF ? 0u : (uint32_t)((n0 % 128) / 32));
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!wait_bounded(&full_bar[s], ph, abort_flag, 13)) goto done;
                    const uint32_t sbase = ring0 + s * C::STAGE_BYTES;
                    const uint64_t adesc = desc_hi | (uint64_t)(sbase >> 4);
                    const uint64_t bdesc = desc_hi | (uint64_t)((sbase + A_BYTES) >> 4);
                    if (elect_one()) {
                        if (MODE == MODE_OSC && kb < nkb_a) {
                            const int ka = min(2, katoms_total - 2 * kb);
                            const uint64_t sfa_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES) >> 4);
                            const uint64_t sfb_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES + C::SFA_BYTES) >> 4);
                            // two scale buffers in TMEM where they fit, alternating by stage (so a stage's copies
                            // never wait for another stage's MMAs still reading theirs)
                            const uint32_t sfo = (uint32_t)(C::SF_BUFS == 2 ? (kb & 1) : 0) * C::TM_SF_STRIDE;
#pragma unroll
                            for (int a = 0; a < 2; ++a) {
                                if (a < ka) {
                                    tc_copy_sf_pair(tmem_base + sfo + C::TM_SFA + a * 4, sfa_d + (uint64_t)(a * 32));
#pragma unroll
                                    for (int j = 0; j < C::SFB_ATOMS; ++j)
                                        tc_copy_sf_pair(tmem_base + sfo + C::TM_SFB + a * (C::SFB_ATOMS * 4) + j * 4,
                                                        sfb_d + (uint64_t)(j * 64 + a * 32));
                                }
                            }
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                if (k < 2 * ka) {
                                    constexpr uint32_t SFID[2] = {idesc_sf_ids(0, 0), idesc_sf_ids(2, 2)};
                                    mma_mxf4_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A | SFID[k & 1],
                                                  tmem_base + sfo + C::TM_SFA + (k >> 1) * 4,
                                                  sfb_tm + sfo + (k >> 1) * (C::SFB_ATOMS * 4), (kb | k) ? 1u : 0u);
                                }
                            }
                        } else if (MODE == MODE_NVF4 && kb < nkb_a) {
                            // four 64-channel scale blocks per stage, one per K = 64 instruction (a whole scale column)
                            const int ka = min(4, katoms_total - 4 * kb);
                            const uint64_t sfa_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES) >> 4);
                            const uint64_t sfb_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES + C::SFA_BYTES) >> 4);
                            const uint32_t sfo = (uint32_t)(C::SF_BUFS == 2 ? (kb & 1) : 0) * C::TM_SF_STRIDE;
#pragma unroll
                            for (int h = 0; h < 4 / C::KA_T; ++h) {   // KA_T blocks in TMEM at a time (all four, or two by two)
#pragma unroll
                                for (int t = 0; t < C::KA_T; ++t) {
                                    const int a = h * C::KA_T + t;
                                    if (a < ka) {
                                        tc_copy_sf_pair(tmem_base + sfo + C::TM_SFA + t * 4, sfa_d + (uint64_t)(a * 32));
#pragma unroll
                                        for (int j = 0; j < C::SFB_ATOMS; ++j)
                                            tc_copy_sf_pair(tmem_base + sfo + C::TM_SFB + t * (C::SFB_ATOMS * 4) + j * 4,
                                                            sfb_d + (uint64_t)(j * (C::KA * 32) + a * 32));
                                    }
                                }
#pragma unroll
                                for (int t = 0; t < C::KA_T; ++t) {
                                    const int k = h * C::KA_T + t;
                                    if (k < ka)
                                        mma_nvf4_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A,
                                                      tmem_base + sfo + C::TM_SFA + t * 4,
                                                      sfb_tm + sfo + t * (C::SFB_ATOMS * 4), (kb | k) ? 1u : 0u);
                                }
                            }
                        } else if (C::DUAL) {
#pragma unroll
                            for (int k = 0; k < 4; ++k) mma_f16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_B, 1u);
                        } else if (MODE == MODE_MXF8) {
                            // one 128-channel scale block per stage: four K = 32 instructions, scale byte k of the column
                            const uint64_t sfa_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES) >> 4);
                            const uint64_t sfb_d = sf_hi | (uint64_t)((sbase + A_BYTES + C::B_BYTES + C::SFA_BYTES) >> 4);
                            const uint32_t sfo = (uint32_t)(C::SF_BUFS == 2 ? (kb & 1) : 0) * C::TM_SF_STRIDE;
                            tc_copy_sf_pair(tmem_base + sfo + C::TM_SFA, sfa_d);
#pragma unroll
                            for (int j = 0; j < C::SFB_ATOMS; ++j)
                                tc_copy_sf_pair(tmem_base + sfo + C::TM_SFB + j * 4, sfb_d + (uint64_t)(j * 32));
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                mma_mxf8_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A | idesc_sf_ids(k, k),
                                              tmem_base + sfo + C::TM_SFA, sfb_tm + sfo, (kb | k) ? 1u : 0u);
                        } else {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                mma_f8_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC_A, (kb | k) ? 1u : 0u);
                        }
                        tc_commit_pair(&empty_bar[s], 3);  // frees the stage in both CTAs
                    }
                    __syncwarp();
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (elect_one()) tc_commit_pair(&tfull_bar[acc], 3);    // accumulator ready in both CTAs
                __syncwarp();
                if (++acc == ACC) {
                    acc = 0;
                    acc_ph ^= 1u;
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (both CTAs)
        // Two warps per TMEM lane quarter (32 accumulator rows), each draining every other 64-column
        // slice: TMEM -> registers -> bf16 -> the warp's swizzled staging tile (32 or 16 rows x 128 bytes) ->
        // TMA store, slice by slice; the stores drain to global memory while the next tile's MMAs run.
        // (Per-thread global stores, 32 rows x 16 bytes per instruction, kept the memory pipe busy and
        // stalled the next tile's MMA issue.)
        const int q = warp & 3;                          // TMEM lane quarter this warp may read
        const uint64_t y_policy = l2_policy_evict_first();
        const int half = (warp - C::EPI_FIRST_WARP) >> 2;  // which of the two warps of that quarter
        int acc = 0;
        uint32_t acc_ph = 0;
        const uint32_t tempty0 = map_to_cta(smem_u32(&tempty_bar[0]), 0);
        // the staging area is shared out evenly: 32, 16 or 8 rows of 128 bytes per warp and pass
        constexpr int WARP_STAGE_BYTES = GU ? 16 * 64 : C::EPI_BYTES / EW;
        uint8_t* stage_buf = smem + STAGES * C::STAGE_BYTES + (half * 4 + q) * WARP_STAGE_BYTES;
        for (int t = pair_id; t < total; t += num_pairs) {
            const Tile ti = tile_of(t);
            const int n0 = ti.n0;
            const int wrow0 = ti.row0 + (int)rank * BM + q * 32;  // first row of this warp
            const int row = wrow0 + lane;
            // FP8 scales, fetched before the wait so that their latency hides behind the K loop: the row's
            // activation scale, and per slice one coalesced load of the 64 weight scales (lane l holds
            // columns 2l, 2l+1; the conversion loop below broadcasts them with shuffles)
            float sxr = 1.0f;
            float2 wsc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            if (MODE == MODE_FP8) {
                if (row < ti.row_end) sxr = args.sx[row];
                const float* swp = args.sw + (int64_t)ti.expert * N;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int col = n0 + (half + u * (EW / 4)) * 64 + 2 * lane;
                    if (half + u * (EW / 4) < C::SLICES && col + 1 < N)
                        wsc[u] = *reinterpret_cast<const float2*>(swp + col);
                }
            }
            if (!wait_bounded(&tfull_bar[acc], acc_ph, abort_flag, 14)) goto done;
            tc_fence_after();
            if (GU) {
                // h = silu(gate) * up for the tile's BN/2 features in chunks of 32 (the last one narrower): this warp
                // takes chunk `half` of its lane quarter.  Staging tile: 16 rows x 64 bytes with the 64-byte swizzle of
                // the store's descriptor, two passes.
                const int I = N >> 1;
                const int f0 = (n0 / BN) * (BN / 2);
                uint8_t* buf = stage_buf;
                const int c0 = half * 32;                            // first feature of the chunk inside the tile
                const int col = f0 + c0;                             // first column of the chunk in H
                if (c0 < BN / 2) {
                    const int wd = min(32, BN / 2 - c0);
                    uint32_t rg[32], ru[32];
                    const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * C::ACC_STRIDE);
                    tmem_ld_32x32(tbase + c0, rg);                   // (a narrow chunk reads past its columns: ignored below)
                    tmem_ld_32x32(tbase + BN / 2 + c0, ru);
                    tmem_ld_wait();
                    if (col < I) {
                        uint4 pk[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t o[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int x = j * 8 + 2 * i;
                                // the projection's outputs as the unfused path stores them: bf16, nearest even
                                const uint32_t g2 = bf162_bits(__floats2bfloat162_rn(__uint_as_float(rg[x]), __uint_as_float(rg[x + 1])));
                                const uint32_t u2 = bf162_bits(__floats2bfloat162_rn(__uint_as_float(ru[x]), __uint_as_float(ru[x + 1])));
                                const float2 h2 = swiglu32x2(make_float2(__uint_as_float(g2 << 16), __uint_as_float(g2 & 0xFFFF0000u)),
                                                             make_float2(__uint_as_float(u2 << 16), __uint_as_float(u2 & 0xFFFF0000u)));
                                o[i] = bf162_bits(__floats2bfloat162_rn(h2.x, h2.y));
                            }
                            pk[j] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            if (lane == 0) tma_store_wait_read<0>();     // the staging tile must be free again
                            __syncwarp();
                            if ((lane >> 4) == hh) {
                                const int rl = lane & 15;
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    *reinterpret_cast<uint4*>(buf + rl * 64 + ((j ^ ((rl >> 1) & 3)) << 4)) = pk[j];
                            }
                            fence_proxy_async_smem();
                            __syncwarp();
                            const int prow0 = wrow0 + hh * 16;
                            // grouped problems: rows past the expert's end belong to the next expert
                            if (wd == 32 && !(sched != nullptr && prow0 + 16 > ti.row_end)) {
                                if (lane == 0) {
                                    tma_store_2d_hint(&args.tm_y16, buf, col, prow0, y_policy);   // clipped at M rows, I columns
                                    tma_store_commit();
                                }
                            } else {
                                // the narrow last chunk is no store box (its neighbours belong to the next tile), nor is a
                                // pass that straddles an expert's end: row-masked 16-byte stores from the staged tile
                                const int j4 = lane & 3;
#pragma unroll
                                for (int rr = 0; rr < 2; ++rr) {
                                    const int rl = rr * 8 + (lane >> 2);
                                    if (prow0 + rl < ti.row_end && j4 * 8 < wd && col + j4 * 8 < I)
                                        *reinterpret_cast<uint4*>(args.Y + (int64_t)(prow0 + rl) * args.ldy + col + j4 * 8) =
                                            *reinterpret_cast<const uint4*>(buf + rl * 64 + ((j4 ^ ((rl >> 1) & 3)) << 4));
                                }
                                __syncwarp();
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(tempty0 + (uint32_t)acc * 8u);
                __syncwarp();
                if (++acc == ACC) { acc = 0; acc_ph ^= 1u; }
                continue;
            }
            // grouped problems: rows past the expert's end belong to the next expert and must not be written,
            // so a warp whose 32 rows straddle the end writes its staged tiles with row-masked stores
            const bool clip = sched != nullptr && wrow0 + 32 > ti.row_end;
            int ord = 0;
#pragma unroll 1
            for (int c = half; c < C::SLICES; c += EW / 4, ++ord) {
                uint32_t r0[32], r1[32];
                const float2 wv = ord == 0 ? wsc[0] : wsc[1];
                const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * C::ACC_STRIDE + c * 64);
                const bool narrow = (C::LAST_W != 64) && (c == C::SLICES - 1);  // last slice of a 240-wide tile: 48 columns
                tmem_ld_32x32(tcol, r0);
                if (narrow) tmem_ld_32x16(tcol + 32, r1); else tmem_ld_32x32(tcol + 32, r1);
                tmem_ld_wait();
                const int col = n0 + c * 64;
                uint8_t* buf = stage_buf;
                if (col < N) {
                    uint4 pk[8];   // the row's 64 outputs as bf16: 8 chunks of 16 bytes = 8 columns each
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t o[4] = {0u, 0u, 0u, 0u};
                        if (!(narrow && j >= C::LAST_W / 8)) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int cc = j * 8 + 2 * i;  // column inside the 64-column slice
                                float lo = __uint_as_float(cc < 32 ? r0[cc] : r1[cc - 32]);
                                float hi = __uint_as_float(cc < 32 ? r0[cc + 1] : r1[cc - 31]);
                                if (MODE == MODE_NVF4) {   // back out of the scaled domain: an exact power of two
                                    lo *= args.out_scale;
                                    hi *= args.out_scale;
                                }
                                if (MODE == MODE_FP8) {
                                    const float wx = __shfl_sync(0xFFFFFFFFu, wv.x, j * 4 + i);
                                    const float wy = __shfl_sync(0xFFFFFFFFu, wv.y, j * 4 + i);
                                    lo = lo * (sxr * wx);
                                    hi = hi * (sxr * wy);
                                }
                                const __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                                o[i] = *reinterpret_cast<const uint32_t*>(&b2);
                            }
                        }
                        pk[j] = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                    constexpr int RPH = WARP_STAGE_BYTES / 128, HV = 32 / RPH;   // rows per pass, staging passes per slice
                    static_assert(GU || HV == 1 || HV == 2, "store boxes of 32 or 16 rows");
#pragma unroll
                    for (int hh = 0; hh < HV; ++hh) {
                        if (lane == 0) tma_store_wait_read<0>();  // the one staging tile must be free again
                        __syncwarp();
                        if (HV == 1 || (lane / RPH) == hh) {
                            const int rl = lane % RPH;
                            // 128-byte swizzle: 16-byte chunk j of row rl lives at chunk j ^ (rl % 8)
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<uint4*>(buf + rl * 128 + ((j ^ (rl & 7)) << 4)) = pk[j];
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        const int prow0 = wrow0 + hh * RPH;   // first output row of this pass
                        if (!clip && !narrow) {
                            if (lane == 0) {
                                tma_store_2d_hint(HV == 1 ? &args.tm_y : &args.tm_y16, buf, col, prow0, y_policy);
                                tma_store_commit();
                            }
                        } else {
                            // rows past the expert's end must stay untouched, and the 48-column last slice of a 240-wide
                            // tile is no TMA box: row-masked 16-byte stores from the staged tile
                            const int j8 = lane & 7;
#pragma unroll
                            for (int rr = 0; rr < RPH / 4; ++rr) {
                                const int rl = rr * 4 + (lane >> 3);
                                if (prow0 + rl < ti.row_end && col + j8 * 8 < N && (!narrow || j8 < C::LAST_W / 8))
                                    *reinterpret_cast<uint4*>(args.Y + (int64_t)(prow0 + rl) * args.ldy + col + j8 * 8) =
                                        *reinterpret_cast<const uint4*>(buf + rl * 128 + ((j8 ^ (rl & 7)) << 4));
                            }
                            __syncwarp();
                        }
                    }
                }
            }
            // accumulator drained: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tempty0 + (uint32_t)acc * 8u);
            __syncwarp();
            if (++acc == ACC) { acc = 0; acc_ph ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all<0>();
        __syncwarp();
    }

done:
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    // neither CTA may leave (or free TMEM) while the other can still touch its shared memory or barriers
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// Tiles are handed out band by band: inside a band of `band` row tiles the pairs walk down the rows of
// one column of weight tiles before moving to the next column, so a weight tile is fetched from HBM once
// per band and the band's activation tiles are fetched once and then served by L2 for every column.  The
// taller the band the fewer times the weights cross HBM, as long as the band's activations stay in L2
// while the columns go by: on B200 (gate_up, M=8192: 4 / 8 / 16 / 32 tiles -> 381 / 365 / 357 / 349 us)
// the gain holds up to about 24 MB of activations per band and turns into a loss beyond it (FP8 down
// projection, 2.8 MB per tile: 16 -> 32 tiles, 366 -> 382 us).
template <int MODE>
static int band_height(const GemmArgs& a) {
    static const int forced = [] { const char* e = getenv("OSC_BAND"); return e ? atoi(e) : 0; }();
    if (forced > 0) return forced;
    const long row_bytes = (MODE == MODE_FP8 || MODE == MODE_MXF8) ? (long)a.K : (long)a.K / 2 + 2L * a.Kop;
    const long tile_bytes = 2L * BM * row_bytes;
    const long fit = (24L << 20) / (tile_bytes > 0 ? tile_bytes : 1);
    return fit < 4 ? 4 : fit > 32 ? 32 : (int)fit;
}

template <int MODE, int BN, bool GU = false>
static cudaError_t launch_cfg(const GemmArgs& a, cudaStream_t st) {
    using C = Cfg<MODE, BN>;
    static PerDevice configured, resident;
    if (cudaError_t e = opt_in_shared_memory(configured, gemm_pair_kernel<MODE, BN, GU>, C::SMEM_BYTES)) return e;
    const int total = a.sched2 ? a.num_sms : ((a.M + 2 * BM - 1) / (2 * BM)) * ((a.N + BN - 1) / BN);
    if (total <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(pair_threads(GU));
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    // The kernel is persistent with static striping of tiles over pairs, so every pair must be
    // resident at once: ask how many 2-CTA clusters of this footprint the device can hold.
    const int slot = per_device_slot();
    int max_pairs = (slot >= 0 && resident.done[slot]) ? resident.value[slot].load() : 0;
    if (max_pairs == 0) {
        cfg.gridDim = dim3(a.num_sms);
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel<MODE, BN, GU>, &cfg);
        if (e != cudaSuccess) return e;
        max_pairs = n > 0 ? n : 1;
        if (slot >= 0) { resident.value[slot] = max_pairs; resident.done[slot] = true; }
        if (getenv("OSC_LOG")) fprintf(stderr, "[osc] pair kernel BN=%d: %d resident clusters of 2\n", BN, max_pairs);
    }
    int pairs = a.num_sms / 2;
    if (max_pairs < pairs) pairs = max_pairs;
    if (const char* e = getenv("OSC_PAIRS")) { const int v = atoi(e); if (v > 0 && v < pairs) pairs = v; }
    if (total < pairs) pairs = total;
    cfg.gridDim = dim3(2 * pairs);
    GemmArgs b = a;
    b.band = band_height<MODE>(a);
    return cudaLaunchKernelEx(&cfg, gemm_pair_kernel<MODE, BN, GU>, b);
}

}  // namespace pair

// Tile width of the pair kernel for a given problem.  The pair tile is 256 x BN and the kernel is
// persistent over num_sms/2 pairs, so the cost is (rounds of tiles) x (time per tile).  Measured on B200
// a K stage costs the same ~370 ns for 192, 240 and 256 columns (the MMA runs at the 256-column rate
// for all three), so wide tiles win; 240 is the widest that leaves room in TMEM for two accumulators
// plus the scale columns (epilogue hidden behind the next tile's K loop unless that loop is shorter
// than the ~2 us drain), 256 has one accumulator (drain and hand-over exposed, ~2.7 us per tile).
// The FP8 mode needs no scale columns: 256 wide with two accumulators.  OSC_PAIR_BLOCK_N overrides.
int gemm_pair_block_n(bool fp8, bool allow_240, long row_tiles, int N, int stages, int num_sms, long* cost_ns) {
    static const int forced = [] {
        const char* e = getenv("OSC_PAIR_BLOCK_N");
        const int v = e ? atoi(e) : 0;
        return (v == 192 || v == 240 || v == 256) ? v : 0;
    }();
    if (cost_ns) *cost_ns = 0;   // a forced width is never weighed against the other kernel
    if (forced && !((fp8 || !allow_240) && forced == 240)) return forced;
    const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
    const long mt = row_tiles;
    const long loop = 370L * stages;
    const long hidden = loop > 2000 ? loop : 2000;
    long best = -1;
    int best_bn = 256;
    const int cand[3] = {256, 240, 192};
    for (int i = 0; i < 3; ++i) {
        const int bn = cand[i];
        if ((fp8 || !allow_240) && bn == 240) continue;
        const long rounds = (mt * ((N + bn - 1) / bn) + pairs - 1) / pairs;
        const bool two_acc = fp8 || bn != 256;
        const long cost = rounds * (two_acc ? hidden : loop + 2700);
        if (best < 0 || cost < best) { best = cost; best_bn = bn; }
    }
    if (cost_ns) *cost_ns = best;
    return best_bn;
}

cudaError_t launch_gemm_dual_pair(const GemmArgs& a, int bn, cudaStream_t st) {
    if (bn == 192) return pair::launch_cfg<pair::MODE_OSC, 192>(a, st);
    if (bn == 240) return pair::launch_cfg<pair::MODE_OSC, 240>(a, st);
    return pair::launch_cfg<pair::MODE_OSC, 256>(a, st);
}
// gate|up projection with the SwiGLU in the epilogue: a.Y / a.ldy / a.tm_y describe H [M, N/2], a.tm_sfw the
// gate|up arrangement of the per-tile weight scales
cudaError_t launch_gemm_dual_pair_swiglu(const GemmArgs& a, cudaStream_t st) {
    return pair::launch_cfg<pair::MODE_OSC, 240, true>(a, st);
}
cudaError_t launch_gemm_mxf8_pair(const GemmArgs& a, int bn, cudaStream_t st) {
    if (bn == 192) return pair::launch_cfg<pair::MODE_MXF8, 192>(a, st);
    return pair::launch_cfg<pair::MODE_MXF8, 256>(a, st);
}
cudaError_t launch_gemm_nvf4_pair(const GemmArgs& a, int bn, cudaStream_t st) {
    if (bn == 192) return pair::launch_cfg<pair::MODE_NVF4, 192>(a, st);
    if (bn == 240) return pair::launch_cfg<pair::MODE_NVF4, 240>(a, st);
    return pair::launch_cfg<pair::MODE_NVF4, 256>(a, st);
}
cudaError_t launch_gemm_fp8_pair(const GemmArgs& a, int bn, cudaStream_t st) {
    if (bn == 192) return pair::launch_cfg<pair::MODE_FP8, 192>(a, st);
    return pair::launch_cfg<pair::MODE_FP8, 256>(a, st);
}

}  // namespace osc
