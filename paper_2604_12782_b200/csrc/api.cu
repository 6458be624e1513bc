// Host side of the C ABI declared in include/osc.h: validation, handles, TMA descriptors, launches.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/osc.h"
#include "common.cuh"

namespace osc {

static thread_local char t_err[512] = "";

static osc_status fail(osc_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_err, sizeof t_err, fmt, ap);
    va_end(ap);
    if (getenv("OSC_LOG")) fprintf(stderr, "[osc] %s: %s\n", osc_status_string(s), t_err);
    return s;
}
static osc_status cuda_fail(cudaError_t e, const char* what) {
    return fail(OSC_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static size_t align256(size_t x) { return (x + 255u) & ~size_t(255); }

// -------------------------------------------------------------- device facts
struct DeviceInfo {
    bool ok = false;
    int num_sms = 0;
};
static osc_status device_info(DeviceInfo* out) {
    int dev = 0, major = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
    if (major != 10) return fail(OSC_ERR_ARCH, "device %d has compute capability %d.x; this library needs 10.x", dev, major);
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
    out->ok = true;
    out->num_sms = sms;
    return OSC_OK;
}

// ------------------------------------------------------------ TMA descriptors
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_fn() {
    static const EncodeTiledFn fn = [] {   // looked up once; initialisation of a local static is thread-safe
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

// Every 2-D descriptor of the library goes through encode_2d.  The descriptors of a call's activation, scratch and
// output buffers depend on caller pointers and on M, so they are built per call - and a call needs up to six of
// them, at one to two microseconds of driver time each, which paces few-row launches from the host.  A descriptor
// is a pure function of the arguments below (an address and a geometry, no driver object behind it), so each host
// thread remembers the last ones it built: a serving loop that reuses its buffers encodes them once.  The cache is
// thread-local (no lock, nothing shared between threads) and replaces its entries round-robin.
struct MapKey {
    const void* base;
    uint64_t dim0, dim1, stride;
    uint32_t box0, box1;
    int dtype, swizzle, device;
    bool operator==(const MapKey& o) const {
        return base == o.base && dim0 == o.dim0 && dim1 == o.dim1 && stride == o.stride && box0 == o.box0 &&
               box1 == o.box1 && dtype == o.dtype && swizzle == o.swizzle && device == o.device;
    }
};
constexpr int kMapCacheEntries = 64;
struct MapCache {
    MapKey key[kMapCacheEntries];
    CUtensorMap map[kMapCacheEntries];
    int used = 0, next = 0;
};

static osc_status encode_2d(CUtensorMap* tm, CUtensorMapDataType dtype, const void* base, uint64_t dim0, uint64_t dim1,
                            uint64_t stride_bytes, uint32_t box0, uint32_t box1, CUtensorMapSwizzle swizzle,
                            const char* what) {
    static thread_local MapCache cache;
    static const bool use_cache = [] { const char* e = getenv("OSC_MAP_CACHE"); return !e || atoi(e) != 0; }();
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
    const MapKey k = {base, dim0, dim1, stride_bytes, box0, box1, (int)dtype, (int)swizzle, dev};
    if (use_cache) {
        for (int i = 0; i < cache.used; ++i)
            if (cache.key[i] == k) { *tm = cache.map[i]; return OSC_OK; }
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(OSC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t gdim[2] = {dim0, dim1};
    cuuint64_t gstr[1] = {stride_bytes};
    cuuint32_t box[2] = {box0, box1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, dtype, 2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_ERROR_INVALID_CONTEXT && dev >= 0 && cudaSetDevice(dev) == cudaSuccess) {
        // The encoder is a driver call and wants a current context.  A host thread that has made no CUDA call of its
        // own yet has none (runtime calls bind the primary context lazily, a bare driver call does not): the primary
        // context of the thread's current device is made current and the call is repeated once.
        r = fn(tm, dtype, 2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return fail(OSC_ERR_CUDA, "cuTensorMapEncodeTiled(%s) failed with code %d", what, (int)r);
    if (use_cache) {
        const int slot = cache.used < kMapCacheEntries ? cache.used++ : (cache.next = (cache.next + 1) % kMapCacheEntries);
        cache.key[slot] = k;
        cache.map[slot] = *tm;
    }
    return OSC_OK;
}

// Row-major [rows, row_bytes] operand, tiles of box_rows x 128 bytes, 128-byte swizzle, zero fill.
static osc_status make_tmap(CUtensorMap* tm, const void* base, bool bf16, uint64_t rows, uint64_t row_bytes,
                            uint64_t pitch_bytes, uint32_t box_rows) {
    if (rows == 0) rows = 1;  // never dereferenced: no tile is scheduled for an empty operand
    const uint64_t esz = bf16 ? 2 : 1;
    return encode_2d(tm, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, base, row_bytes / esz, rows,
                     pitch_bytes, static_cast<uint32_t>(128 / esz), box_rows, CU_TENSOR_MAP_SWIZZLE_128B, "operand");
}

// bf16 [rows, cols] input of the quantizer: tiles of 128 rows x 64 channels (128 bytes), 128-byte swizzle, zero fill.
static osc_status make_tmap_x(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
    if (rows == 0) rows = 1;
    return encode_2d(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, cols, rows, ld * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B, "X");
}

// Scale-factor buffer as [blocks, 128] uint32 (512-byte blocks), tiles of `box_blocks` consecutive blocks
// (2 = the 256 FP4 channels of a GEMM stage, 1 = the 128 FP8 channels).
static osc_status make_tmap_sf(CUtensorMap* tm, const void* base, uint64_t blocks, uint32_t box_blocks = 2) {
    if (blocks == 0) blocks = 1;
    return encode_2d(tm, CU_TENSOR_MAP_DATA_TYPE_UINT32, base, 128, blocks, 512, 128, box_blocks, CU_TENSOR_MAP_SWIZZLE_NONE,
                     "scales");
}

// Grouped problems whose experts average at least 96 rows run on the CTA-pair kernel (256-row tiles), the rest on
// the single-CTA kernel (128-row tiles).  Dense problems with more than 128 rows take whichever kernel its cost
// model puts ahead (single_ns / pair_ns: estimated time of the whole K loop over all waves of tiles): the pair
// kernel is more than twice as efficient per tile, but with few rows and a long K loop its tiles fill a fraction
// of the machine - down projection 12288 -> 4096 with 256 rows: 16 pair tiles on 74 pairs, 38 us, against 128
// single-CTA tiles of 128 x 64 in one wave, 27 us.  The single-CTA estimate only holds while all its tiles run in
// one wave (with more, the SMs compete for the L2 feed and it is about half as fast as the pair kernel), so it is
// only considered then.  OSC_PAIR=0: never, OSC_PAIR=2: always when eligible.
static bool use_pair_kernel(bool grouped, int M, int E, long single_ns = 0, long pair_ns = 0, bool single_one_wave = false) {
    static const int mode = [] {
        const char* e = getenv("OSC_PAIR");
        const int v = e ? atoi(e) : 1;
        return (v < 0 || v > 2) ? 1 : v;
    }();
    if (mode == 0) return false;
    if (grouped) return M / E >= 96;
    if (M <= 128) return false;
    if (mode == 2 || single_ns <= 0 || pair_ns <= 0) return true;
    return !single_one_wave || pair_ns <= single_ns;
}

// Dense problems with few rows run on the few-row kernel (operands swapped, K split over a cluster): up to 32
// rows always; up to 64 rows when there are more 128-feature tiles than SMs or the K loop is long (64 stages or
// more) - measured on B200: with 48 tiles, 20 stages and 64 rows the 128-row-tile kernel is still ahead (11.5 vs
// 14.4 us), with 32 tiles and 96 stages it is behind (24.4 vs 21.9 us); up to 256 rows (its 256-token form, one
// CTA per SM) when the K loop is long and the tiles with their K split still fit the machine, where the tile
// kernels leave most SMs idle.  OSC_DECODE=0 disables, OSC_DECODE=2 forces it up to 256 rows.
// no_row128: the format has no 128-row-tile kernel (NVFP4), so up to 64 rows the alternative is the pair kernel with
// three quarters of its tile empty: QKV / gate_up / o_proj at 64 rows 10.9 / 19.3 / 10.5 us against 13.8 / 22.9 / 13.6.
static bool use_decode_kernel(bool grouped, int M, int N, int nkb, int num_sms, bool no_row128 = false) {
    const char* e = getenv("OSC_DECODE");   // read per call: tests switch it inside one process
    const int mode = e ? atoi(e) : 1;
    if (mode == 0 || grouped || M > 256) return false;
    if (mode == 2) return true;
    const int tiles = (N + 127) / 128;
    if (M <= 32) return true;
    if (M <= 64) return no_row128 || tiles >= num_sms || nkb >= 64;
    return nkb >= 64 && 2 * tiles <= num_sms;
}

// ----------------------------------------------------------------- the table
struct Table {
    int Ko = 0, Kop = 0;
    std::vector<uint32_t> mask;
    std::vector<int32_t> prefix, idx;
};
static osc_status parse_lut(const int8_t* lut, int K, int C, Table* t) {
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    if (C < 0 || C > 32) return fail(OSC_ERR_INVALID_ARG, "lut_c = %d outside 0..32", C);
    if (C > 0 && !lut) return fail(OSC_ERR_INVALID_ARG, "lut is null");
    const int Kg = K / 32;
    t->mask.assign(Kg, 0);
    t->prefix.assign(Kg, 0);
    t->idx.clear();
    for (int k = 0; k < Kg; ++k) {
        uint32_t m = 0;
        for (int c = 0; c < C; ++c) {
            const int j = lut[(size_t)k * C + c];
            if (j < -1 || j > 31) return fail(OSC_ERR_LUT, "table entry %d of group %d outside -1..31", j, k);
            if (j < 0) continue;
            if (m >> j & 1u) return fail(OSC_ERR_LUT, "channel %d listed twice in group %d", j, k);
            m |= 1u << j;
        }
        t->mask[k] = m;
        t->prefix[k] = (int32_t)t->idx.size();
        for (int j = 0; j < 32; ++j)
            if (m >> j & 1u) t->idx.push_back(k * 32 + j);
    }
    t->Ko = (int)t->idx.size();
    t->Kop = (t->Ko + 63) / 64 * 64;
    return OSC_OK;
}

static osc_status check_nk(int E, int N, int K) {
    if (E < 1 || E > 1024) return fail(OSC_ERR_INVALID_ARG, "E = %d outside 1..1024", E);
    if (N <= 0 || N % 64) return fail(OSC_ERR_SHAPE, "N = %d must be a positive multiple of 64", N);
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    if ((int64_t)E * N > 0x7FFFFFFF) return fail(OSC_ERR_SHAPE, "E*N too large");
    return OSC_OK;
}
static size_t sf_bytes(int64_t rows, int K) { return (size_t)((rows + 127) / 128) * (K / 128) * 512; }
// meta = [mask | prefix | idx_o, padded to 1 KB][per-tile copy of the weight scales for 240-row tiles (dense only)]
constexpr int kTiledBN = 240;
static size_t meta_table_bytes(int K, int Ko) { return ((size_t)(K / 32) * 8 + (size_t)Ko * 4 + 16 + 1023) & ~size_t(1023); }
static size_t tiled_sf_bytes(int N, int K) {
    return (size_t)((N + kTiledBN - 1) / kTiledBN) * ((kTiledBN + 127) / 128) * (K / 128) * 512;
}

}  // namespace osc

using namespace osc;

struct osc_weights {
    int E, N, K, Ko, Kop;
    bool grouped;
    bool dynamic;   // weights of the dynamic-protection control group: whole-matrix MXFP4 + the bf16 matrix (Kop = K)
    bool nvfp4;     // NVFP4 / G = 16 variant: E4M3 block scales per 16 channels, tensor-level scale 2^ew
    int ew;
    const uint8_t *wq, *sfw;
    const uint16_t* wo;
    const uint32_t* mask;
    const int32_t* prefix;
    const int32_t* idx_o;
    int num_sms;
    CUtensorMap tm_b[4], tm_bo[4];    // single-CTA kernel: weight tiles of 64 / 128 / 192 / 256 rows
    CUtensorMap tm_b2[3], tm_bo2[3];  // CTA-pair kernel: half tiles for 192-, 256- and 240-wide tiles
    CUtensorMap tm_sfw, tm_sfw_tiled;  // scale blocks: standard layout / per-tile copy for 240-wide tiles
    bool gate_up;                      // prepared by osc_prepare_weights_gate_up: rows [0, N/2) gate, [N/2, N) up
    CUtensorMap tm_sfw_gu;             // per-tile copy of the scales in the gate|up arrangement of a tile
};
struct osc_fp8_weights {
    int E, N, K;
    bool grouped;
    const uint8_t* w8;
    const float* sw;
    int num_sms;
    CUtensorMap tm_b[4], tm_b2[2];
};

struct osc_mxfp8_weights {
    int E, N, K;
    bool grouped;
    const uint8_t *w8, *sfw;
    int num_sms;
    CUtensorMap tm_b2[2];  // half tiles for 192- and 256-wide tiles
    CUtensorMap tm_b128;   // 128-row weight tiles of the few-row kernel
    CUtensorMap tm_b1[4];  // single-CTA kernel: 64-, 128-, 192- and 256-row weight tiles
    CUtensorMap tm_sfw;
};

extern "C" {

const char* osc_status_string(osc_status s) {
    switch (s) {
        case OSC_OK: return "OSC_OK";
        case OSC_ERR_INVALID_ARG: return "OSC_ERR_INVALID_ARG";
        case OSC_ERR_SHAPE: return "OSC_ERR_SHAPE";
        case OSC_ERR_LUT: return "OSC_ERR_LUT";
        case OSC_ERR_ALIGN: return "OSC_ERR_ALIGN";
        case OSC_ERR_WORKSPACE: return "OSC_ERR_WORKSPACE";
        case OSC_ERR_ARCH: return "OSC_ERR_ARCH";
        case OSC_ERR_CUDA: return "OSC_ERR_CUDA";
        case OSC_ERR_TIMEOUT: return "OSC_ERR_TIMEOUT";
        default: return "OSC_ERR_UNKNOWN";
    }
}
const char* osc_last_error(void) { return t_err; }

osc_status osc_sync_check(void* stream) {
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    int st = 0;
    e = cudaMemcpyFromSymbol(&st, g_dev_status, sizeof st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyFromSymbol");
    if (st != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_dev_status, &zero, sizeof zero);
        return fail(OSC_ERR_TIMEOUT, "a device-side wait gave up (site %d)", st >> 8);
    }
    return OSC_OK;
}

// ------------------------------------------------------------------ OSC path

osc_status osc_weight_sizes(int E, int N, int K, const int8_t* lut, int lut_c, osc_weight_sizes_t* out) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    if (osc_status s = check_nk(E, N, K)) return s;
    Table t;
    if (osc_status s = parse_lut(lut, K, lut_c, &t)) return s;
    out->K_o = t.Ko;
    out->K_o_pad = t.Kop;
    out->wq_bytes = (size_t)E * N * (K / 2);
    out->sfw_bytes = (size_t)E * sf_bytes(N, K);
    out->wo_bytes = (size_t)E * N * t.Kop * 2;
    out->meta_bytes = meta_table_bytes(K, t.Ko) + (E == 1 ? tiled_sf_bytes(N, K) : 0);
    return OSC_OK;
}

static osc_status prepare_impl(const void* W, int E, int N, int K, int64_t ldw, const int8_t* lut, int lut_c,
                               void* wq, void* sfw, void* wo, void* meta, void* stream, bool grouped,
                               osc_weights** out, bool dynamic = false, bool gate_up = false) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if (osc_status s = check_nk(E, N, K)) return s;
    Table t;
    if (osc_status s = parse_lut(lut, K, lut_c, &t)) return s;
    if (!W || !wq || !sfw || !meta || ((t.Kop > 0 || dynamic) && !wo)) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldw < K) return fail(OSC_ERR_SHAPE, "ldw = %lld < K", (long long)ldw);
    if (ldw % 8 || !aligned16(W) || !aligned16(wq) || !aligned16(sfw) || !aligned16(meta) || !aligned16(wo))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldw a multiple of 8");
    DeviceInfo di;
    if (osc_status s = device_info(&di)) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const int Kg = K / 32;
    uint8_t* m8 = static_cast<uint8_t*>(meta);
    cudaError_t e = cudaMemcpyAsync(m8, t.mask.data(), (size_t)Kg * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(m8 + (size_t)Kg * 4, t.prefix.data(), (size_t)Kg * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && t.Ko > 0)
        e = cudaMemcpyAsync(m8 + (size_t)Kg * 8, t.idx.data(), (size_t)t.Ko * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(meta)");
    const uint32_t* d_mask = reinterpret_cast<const uint32_t*>(m8);
    const int32_t* d_prefix = reinterpret_cast<const int32_t*>(m8 + (size_t)Kg * 4);

    const size_t sfw_e = sf_bytes(N, K);
    for (int ex = 0; ex < E; ++ex) {
        CUtensorMap tm_w;
        if (osc_status s = make_tmap_x(&tm_w, static_cast<const uint16_t*>(W) + (size_t)ex * N * ldw, N, K, ldw)) return s;
        e = launch_quant_extract(tm_w, N, K, d_mask, d_prefix, reinterpret_cast<const int32_t*>(m8 + (size_t)Kg * 8),
                                 static_cast<uint8_t*>(wq) + (size_t)ex * N * (K / 2),
                                 static_cast<uint8_t*>(sfw) + (size_t)ex * sfw_e,
                                 t.Kop ? static_cast<uint16_t*>(wo) + (size_t)ex * N * t.Kop : nullptr, t.Ko, t.Kop,
                                 nullptr, 0, di.num_sms, st);
        if (e != cudaSuccess) return cuda_fail(e, "quant_extract_kernel(weights)");
    }

    const size_t tiled_off = meta_table_bytes(K, t.Ko);   // the per-tile scale copy follows the table
    if (dynamic) {
        // the high-precision operand is the bf16 matrix itself, compacted to [N, K]; from here on the handle
        // looks like one whose table lists every channel, except that no column was zeroed before quantization
        e = cudaMemcpy2DAsync(wo, (size_t)K * 2, W, (size_t)ldw * 2, (size_t)K * 2, (size_t)N, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy2DAsync(weights)");
        t.Ko = t.Kop = K;
    }
    osc_weights* w = new (std::nothrow) osc_weights();
    if (!w) return fail(OSC_ERR_INVALID_ARG, "out of host memory");
    w->E = E; w->N = N; w->K = K; w->Ko = t.Ko; w->Kop = t.Kop; w->grouped = grouped; w->dynamic = dynamic;
    w->wq = static_cast<const uint8_t*>(wq);
    w->sfw = static_cast<const uint8_t*>(sfw);
    w->wo = static_cast<const uint16_t*>(wo);
    w->mask = d_mask; w->prefix = d_prefix;
    w->idx_o = reinterpret_cast<const int32_t*>(m8 + (size_t)Kg * 8);
    w->num_sms = di.num_sms;
    osc_status s = OSC_OK;
    for (int v = 0; v < 4 && s == OSC_OK; ++v) {
        s = make_tmap(&w->tm_b[v], wq, false, (uint64_t)E * N, K / 2, K / 2, 64 * (v + 1));
        if (s == OSC_OK && t.Kop > 0)
            s = make_tmap(&w->tm_bo[v], wo, true, (uint64_t)E * N, (uint64_t)t.Kop * 2, (uint64_t)t.Kop * 2, 64 * (v + 1));
    }
    for (int v = 0; v < 3 && s == OSC_OK; ++v) {
        if (grouped && v == 2 && !gate_up) break;  // 240-wide tiles need a per-tile scale copy: dense weights, or gate|up
        const int half = (v == 0 ? 192 : v == 1 ? 256 : kTiledBN) / 2;
        s = make_tmap(&w->tm_b2[v], wq, false, (uint64_t)E * N, K / 2, K / 2, half);
        if (s == OSC_OK && t.Kop > 0)
            s = make_tmap(&w->tm_bo2[v], wo, true, (uint64_t)E * N, (uint64_t)t.Kop * 2, (uint64_t)t.Kop * 2, half);
    }
    if (s == OSC_OK) s = make_tmap_sf(&w->tm_sfw, sfw, (uint64_t)E * sfw_e / 512);
    if (s == OSC_OK && !grouped) {
        uint8_t* tiled = m8 + tiled_off;
        e = launch_retile_sf(static_cast<const uint8_t*>(sfw), tiled, N, K, kTiledBN, st);
        if (e != cudaSuccess) { delete w; return cuda_fail(e, "retile_sf_kernel"); }
        s = make_tmap_sf(&w->tm_sfw_tiled, tiled, (uint64_t)tiled_sf_bytes(N, K) / 512);
        if (s == OSC_OK && gate_up) {   // a second copy behind the first, rows of a tile in gate|up order
            uint8_t* tiled_gu = tiled + tiled_sf_bytes(N, K);
            e = launch_retile_sf(static_cast<const uint8_t*>(sfw), tiled_gu, N, K, kTiledBN, st, true);
            if (e != cudaSuccess) { delete w; return cuda_fail(e, "retile_sf_kernel(gate|up)"); }
            s = make_tmap_sf(&w->tm_sfw_gu, tiled_gu, (uint64_t)tiled_sf_bytes(N, K) / 512);
            w->gate_up = true;
        }
    } else if (s == OSC_OK && gate_up) {   // grouped gate|up: one gate|up-ordered per-tile copy per expert, behind the table
        uint8_t* tiled_gu = m8 + tiled_off;
        const size_t per = tiled_sf_bytes(N, K);
        for (int x = 0; x < E; ++x) {
            e = launch_retile_sf(static_cast<const uint8_t*>(sfw) + (size_t)x * sfw_e, tiled_gu + (size_t)x * per, N, K, kTiledBN, st, true);
            if (e != cudaSuccess) { delete w; return cuda_fail(e, "retile_sf_kernel(gate|up, grouped)"); }
        }
        s = make_tmap_sf(&w->tm_sfw_gu, tiled_gu, (uint64_t)E * per / 512);
        w->gate_up = true;
    }
    if (s == OSC_OK && (e = launch_prepare_fence(st)) != cudaSuccess) s = cuda_fail(e, "prepare_fence_kernel");
    if (s != OSC_OK) { delete w; return s; }
    *out = w;
    return OSC_OK;
}

osc_status osc_prepare_weights(const void* W, int N, int K, int64_t ldw, const int8_t* lut, int lut_c, void* wq,
                               void* sfw, void* wo, void* meta, void* stream, osc_weights** out) {
    return prepare_impl(W, 1, N, K, ldw, lut, lut_c, wq, sfw, wo, meta, stream, false, out);
}
osc_status osc_prepare_weights_grouped(const void* W, int E, int N, int K, const int8_t* lut, int lut_c, void* wq,
                                       void* sfw, void* wo, void* meta, void* stream, osc_weights** out) {
    return prepare_impl(W, E, N, K, K, lut, lut_c, wq, sfw, wo, meta, stream, true, out);
}
// ---- gate|up projection with the SwiGLU in the GEMM epilogue
osc_status osc_gate_up_weight_sizes(int I, int K, const int8_t* lut, int lut_c, osc_weight_sizes_t* out) {
    if (I <= 0 || I % 64 || I > (1 << 29)) return fail(OSC_ERR_SHAPE, "I = %d must be a positive multiple of 64", I);
    if (osc_status s = osc_weight_sizes(1, 2 * I, K, lut, lut_c, out)) return s;
    out->meta_bytes += tiled_sf_bytes(2 * I, K);
    return OSC_OK;
}
osc_status osc_prepare_weights_gate_up(const void* W, int I, int K, int64_t ldw, const int8_t* lut, int lut_c, void* wq,
                                       void* sfw, void* wo, void* meta, void* stream, osc_weights** out) {
    if (I <= 0 || I % 64 || I > (1 << 29)) return fail(OSC_ERR_SHAPE, "I = %d must be a positive multiple of 64", I);
    return prepare_impl(W, 1, 2 * I, K, ldw, lut, lut_c, wq, sfw, wo, meta, stream, false, out, false, true);
}
osc_status osc_gate_up_weight_sizes_grouped(int E, int I, int K, const int8_t* lut, int lut_c, osc_weight_sizes_t* out) {
    if (I <= 0 || I % 64 || I > (1 << 29)) return fail(OSC_ERR_SHAPE, "I = %d must be a positive multiple of 64", I);
    if (osc_status s = osc_weight_sizes(E, 2 * I, K, lut, lut_c, out)) return s;
    out->meta_bytes = meta_table_bytes(K, out->K_o) + (size_t)E * tiled_sf_bytes(2 * I, K);
    return OSC_OK;
}
osc_status osc_prepare_weights_gate_up_grouped(const void* W, int E, int I, int K, const int8_t* lut, int lut_c, void* wq,
                                               void* sfw, void* wo, void* meta, void* stream, osc_weights** out) {
    if (I <= 0 || I % 64 || I > (1 << 29)) return fail(OSC_ERR_SHAPE, "I = %d must be a positive multiple of 64", I);
    return prepare_impl(W, E, 2 * I, K, K, lut, lut_c, wq, sfw, wo, meta, stream, true, out, false, true);
}

osc_status osc_weights_destroy(osc_weights* w) {
    delete w;
    return OSC_OK;
}

// A grouped workspace holds two tile schedules, back to back: 128-row tiles (quantizer, single-CTA GEMM) and
// 256-row tiles (CTA-pair GEMM).  Each is 1 + 4 * max_tiles int32, rounded up to 64.
static size_t sched_ints(int64_t max_tiles) { return (size_t)((1 + 4 * max_tiles + 63) / 64 * 64); }
static int max_tiles256(int M, int E) { return M / 256 + E; }

osc_status osc_act_sizes(const osc_weights* w, int M, osc_act_sizes_t* out) {
    if (!w || !out) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (w->nvfp4) return fail(OSC_ERR_INVALID_ARG, "NVFP4 weights: use osc_nvfp4_act_sizes");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    const int64_t max_tiles = w->grouped ? (int64_t)M / 128 + w->E : ((int64_t)M + 127) / 128;
    out->xq_bytes = (size_t)M * (w->K / 2);
    out->sfa_bytes = (size_t)max_tiles * (w->K / 128) * 512;
    out->xo_bytes = (size_t)M * w->Kop * 2;
    out->sched_bytes = w->grouped ? sched_ints(max_tiles) * 4 + sched_ints(max_tiles256(M, w->E)) * 4 : 0;
    out->xq_offset = 0;
    out->sfa_offset = out->xq_offset + align256(out->xq_bytes);
    out->xo_offset = out->sfa_offset + align256(out->sfa_bytes);
    out->sched_offset = out->xo_offset + align256(out->xo_bytes);
    out->workspace_bytes = out->sched_offset + align256(out->sched_bytes);
    return OSC_OK;
}

static osc_status check_act(const osc_weights* w, const void* X, int M, int64_t ldx, bool dynamic = false,
                            bool nvfp4 = false) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (w->nvfp4 != nvfp4)
        return fail(OSC_ERR_INVALID_ARG, nvfp4 ? "MXFP4 weights: use osc_linear" : "NVFP4 weights: use osc_nvfp4_linear");
    if (w->dynamic != dynamic)
        return fail(OSC_ERR_INVALID_ARG, dynamic ? "static-table weights: use osc_linear" : "dynamic-protection weights: use osc_dyn_linear");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (M > 0 && !X) return fail(OSC_ERR_INVALID_ARG, "X is null");
    if (ldx < w->K) return fail(OSC_ERR_SHAPE, "ldx = %lld < K = %d", (long long)ldx, w->K);
    if (ldx % 8 || !aligned16(X)) return fail(OSC_ERR_ALIGN, "X must be 16-byte aligned and ldx a multiple of 8");
    return OSC_OK;
}

static osc_status quantize_impl(const osc_weights* w, const void* X, int M, int64_t ldx, void* xq, void* sfa,
                                void* xo, const int32_t* sched, int max_tiles, cudaStream_t st) {
    if (M == 0) return OSC_OK;
    if (!xq || !sfa || (w->Kop > 0 && !xo)) return fail(OSC_ERR_INVALID_ARG, "null output pointer");
    if (!aligned16(xq) || !aligned16(sfa) || !aligned16(xo)) return fail(OSC_ERR_ALIGN, "outputs must be 16-byte aligned");
    CUtensorMap tm_x;
    if (osc_status s = make_tmap_x(&tm_x, X, M, w->K, ldx)) return s;
    cudaError_t e = launch_quant_extract(tm_x, M, w->K, w->mask, w->prefix, w->idx_o, xq, sfa, w->Kop ? xo : nullptr, w->Ko,
                                         w->Kop, sched, max_tiles, w->num_sms, st);
    if (e != cudaSuccess) return cuda_fail(e, "quant_extract_kernel");
    return OSC_OK;
}

osc_status osc_quantize_extract(const osc_weights* w, const void* X, int M, int64_t ldx, void* xq, void* sfa,
                                void* xo, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_linear_grouped");
    return quantize_impl(w, X, M, ldx, xq, sfa, xo, nullptr, 0, static_cast<cudaStream_t>(stream));
}

static osc_status gemm_impl(const osc_weights* w, const void* xq, const void* sfa, const void* xo, int M, void* Y,
                            int64_t ldy, const int32_t* sched, int max_tiles, const int32_t* sched2, int max_tiles2,
                            cudaStream_t st) {
    if (M == 0) return OSC_OK;
    if (!xq || !sfa || !Y || (w->Kop > 0 && !xo)) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y) || !aligned16(xq) || !aligned16(sfa) || !aligned16(xo))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldy a multiple of 8");
    GemmArgs a;
    memset(&a, 0, sizeof a);
    if (use_decode_kernel(w->grouped, M, w->N, (w->K + 255) / 256 + w->Kop / 64, w->num_sms)) {
        const uint32_t tok_box = (uint32_t)((M + 15) / 16 * 16);   // activation rows per tile = the MMA's N
        if (osc_status s = make_tmap(&a.tm_a, xq, false, M, w->K / 2, w->K / 2, tok_box)) return s;
        a.tm_b = w->tm_b[1];
        if (w->Kop > 0) {
            if (osc_status s = make_tmap(&a.tm_ao, xo, true, M, (uint64_t)w->Kop * 2, (uint64_t)w->Kop * 2, tok_box)) return s;
            a.tm_bo = w->tm_bo[1];
        }
        a.sfa = static_cast<const uint8_t*>(sfa);
        a.sfw = w->sfw;
        a.Y = static_cast<uint16_t*>(Y);
        a.ldy = ldy;
        a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
        a.num_sms = w->num_sms;
        const int S = gemm_decode_split(w->N, (w->K + 255) / 256 + w->Kop / 64, w->num_sms);
        cudaError_t e = launch_gemm_dual_decode(a, S, st);
        if (e != cudaSuccess) return cuda_fail(e, "gemm_decode_kernel(dual)");
        return OSC_OK;
    }
    if (osc_status s = make_tmap(&a.tm_a, xq, false, M, w->K / 2, w->K / 2, 128)) return s;
    const int nkb = (w->K + 255) / 256 + w->Kop / 64;
    long single_ns = 0, pair_ns = 0;
    const int bn1 = gemm_block_n(sched ? max_tiles : (M + 127) / 128, w->N, w->num_sms, &single_ns);
    const long row_tiles2 = w->grouped ? (max_tiles2 > w->E / 2 ? max_tiles2 - w->E / 2 : 1) : (M + 255) / 256;
    const int bn2 = gemm_pair_block_n(false, !w->grouped, row_tiles2, w->N, nkb, w->num_sms, &pair_ns);
    a.tm_b = w->tm_b[bn1 / 64 - 1];
    if (w->Kop > 0) {
        if (osc_status s = make_tmap(&a.tm_ao, xo, true, M, (uint64_t)w->Kop * 2, (uint64_t)w->Kop * 2, 128)) return s;
        a.tm_bo = w->tm_bo[bn1 / 64 - 1];
    }
    a.sfa = static_cast<const uint8_t*>(sfa);
    a.sfw = w->sfw;
    a.Y = static_cast<uint16_t*>(Y);
    a.ldy = ldy;
    a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
    a.sched = sched; a.max_tiles = max_tiles; a.num_sms = w->num_sms;
    a.sched2 = sched2; a.max_tiles2 = max_tiles2;
    cudaError_t e;
    if (use_pair_kernel(w->grouped, M, w->E, single_ns * nkb, pair_ns, single_ns <= 470)) {
        const int bn = bn2;
        const int v = bn == 192 ? 0 : bn == 256 ? 1 : 2;
        a.tm_b = w->tm_b2[v];
        a.tm_bo = w->tm_bo2[v];
        a.tm_sfw = (bn == kTiledBN) ? w->tm_sfw_tiled : w->tm_sfw;
        const uint64_t sf_row_blocks = w->grouped ? (uint64_t)max_tiles : (uint64_t)((M + 127) / 128);
        if (osc_status s = make_tmap_sf(&a.tm_sfa, sfa, sf_row_blocks * (w->K / 128))) return s;
        if (osc_status s = make_tmap(&a.tm_y, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 32)) return s;
        if (osc_status s = make_tmap(&a.tm_y16, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 16)) return s;
        e = launch_gemm_dual_pair(a, bn, st);
    } else {
        e = launch_gemm_dual(a, bn1, st);
    }
    if (e != cudaSuccess) return cuda_fail(e, "gemm_kernel(dual)");
    return OSC_OK;
}

osc_status osc_gemm_dual(const osc_weights* w, const void* xq, const void* sfa, const void* xo, int M, void* Y,
                         int64_t ldy, void* stream) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_linear_grouped");
    if (w->nvfp4) return fail(OSC_ERR_INVALID_ARG, "NVFP4 weights: use osc_nvfp4_gemm");
    return gemm_impl(w, xq, sfa, xo, M, Y, ldy, nullptr, 0, nullptr, 0, static_cast<cudaStream_t>(stream));
}

// With very few rows the quantizer kernel in front of the few-row GEMM costs more than its work: the GEMM kernel's
// CTAs quantize the activations of their own K slice themselves (same arithmetic, same result).  Every feature
// tile repeats that work, one warp per stage, so it pays while (row quarters) x (stages per CTA) stays small -
// measured on B200, graph replay, two kernels -> one: QKV 4096 -> 6144 8.3 / 8.8 / 9.3 -> 6.5 / 7.3 / 8.9 us at 1 / 8 / 16
// rows, o_proj 8.3 / 8.5 -> 5.8 / 7.8 us at 4 / 16 rows, gate_up (18 stages per CTA) 14.4 / 14.6 -> 12.8 / 13.2 us at 1 / 4
// rows but 14.9 -> 16.9 us at 16 rows, K = 12288 with 768 flagged channels 12.6 -> 9.8 us at 4 rows but 13.1 -> 20.5 us
// at 16 (the Path-B blocks are gathered two bytes at a time).  Tables of more than 1024 flagged channels take
// the two kernels.  OSC_DECODE_FUSED_ROWS = 0: always two kernels; = n: the fused form whenever M <= min(n, 16).
static bool decode_quantizes_itself(const osc_weights* w, int M) {
    if (M > 16 || w->Kop > 1024) return false;
    const int nkb = (w->K + 255) / 256 + w->Kop / 64;
    if (!use_decode_kernel(w->grouped, M, w->N, nkb, w->num_sms)) return false;
    if (const char* e = getenv("OSC_DECODE_FUSED_ROWS")) return M <= atoi(e);   // read per call: tests switch it inside one process
    const int S = gemm_decode_split(w->N, nkb, w->num_sms);
    const int quarters = (M + 3) / 4;
    return quarters * ((nkb + S - 1) / S) <= 24 && quarters * (w->Kop / 64) <= 24;
}
static osc_status gemm_decode_quant_impl(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                                         cudaStream_t st) {
    GemmArgs a;
    memset(&a, 0, sizeof a);
    a.tm_b = w->tm_b[1];
    if (w->Kop > 0) a.tm_bo = w->tm_bo[1];
    a.sfw = w->sfw;
    a.Y = static_cast<uint16_t*>(Y);
    a.ldy = ldy;
    a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
    a.num_sms = w->num_sms;
    DecodeX xa;
    xa.X = static_cast<const uint16_t*>(X);
    xa.ldx = ldx;
    xa.mask = w->mask;
    xa.idx_o = w->idx_o;
    xa.Ko = w->Ko;
    const int S = gemm_decode_split(w->N, (w->K + 255) / 256 + w->Kop / 64, w->num_sms);
    cudaError_t e = launch_gemm_dual_decode_quant(a, xa, S, st);
    if (e != cudaSuccess) return cuda_fail(e, "gemm_decode_kernel(dual, quantizing)");
    return OSC_OK;
}

osc_status osc_linear(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                      void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_linear_grouped");
    if (M == 0) return OSC_OK;
    osc_act_sizes_t sz;
    osc_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (decode_quantizes_itself(w, M)) return gemm_decode_quant_impl(w, X, M, ldx, Y, ldy, st);
    if (osc_status s = quantize_impl(w, X, M, ldx, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, nullptr, 0, st)) return s;
    return gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M, Y, ldy, nullptr, 0, nullptr, 0, st);
}

// ---- RMSNorm fused in front of Algorithm 2
// Optional residual update in front of the norm: h' = bf16(h + r), written to Hout.
struct Residual {
    const void* R = nullptr;
    int64_t ldr = 0;
    void* Hout = nullptr;
    int64_t ldo = 0;
};
static osc_status check_residual(const Residual& res, int K) {
    if (!res.R || !res.Hout) return fail(OSC_ERR_INVALID_ARG, "R / Hout is null");
    if (res.ldr < K || res.ldo < K) return fail(OSC_ERR_SHAPE, "ldr = %lld, ldo = %lld < K = %d", (long long)res.ldr, (long long)res.ldo, K);
    if (res.ldr % 8 || res.ldo % 8 || !aligned16(res.R) || !aligned16(res.Hout))
        return fail(OSC_ERR_ALIGN, "R and Hout must be 16-byte aligned, ldr and ldo multiples of 8");
    return OSC_OK;
}

static osc_status rmsnorm_only_impl(const void* H, int M, int K, int64_t ldh, const void* gamma, float eps, void* X,
                                    int64_t ldx, void* stream, const Residual* res) {
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    if (K > 8192) return fail(OSC_ERR_SHAPE, "K = %d: the fused RMSNorm stages a row in shared memory, K <= 8192", K);
    if (M == 0) return OSC_OK;
    if (!H || !gamma || !X) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldh < K || ldx < K) return fail(OSC_ERR_SHAPE, "ldh = %lld, ldx = %lld < K = %d", (long long)ldh, (long long)ldx, K);
    if (ldh % 8 || ldx % 8 || !aligned16(H) || !aligned16(X) || !aligned16(gamma))
        return fail(OSC_ERR_ALIGN, "H, X and gamma must be 16-byte aligned, ldh and ldx multiples of 8");
    if (res) {
        if (osc_status s = check_residual(*res, K)) return s;
    }
    const Residual none;
    const Residual& rs = res ? *res : none;
    cudaError_t e = launch_rmsnorm_quant(false, H, ldh, M, K, gamma, eps, X, ldx, nullptr, nullptr, nullptr, nullptr,
                                         0, 0, static_cast<cudaStream_t>(stream), rs.R, rs.ldr, rs.Hout, rs.ldo);
    if (e != cudaSuccess) return cuda_fail(e, "rmsnorm_quant_kernel(norm only)");
    return OSC_OK;
}

osc_status osc_rmsnorm(const void* H, int M, int K, int64_t ldh, const void* gamma, float eps, void* X, int64_t ldx,
                       void* stream) {
    return rmsnorm_only_impl(H, M, K, ldh, gamma, eps, X, ldx, stream, nullptr);
}
osc_status osc_add_rmsnorm(const void* H, const void* R, int M, int K, int64_t ldh, int64_t ldr, const void* gamma, float eps,
                           void* Hout, int64_t ldo, void* X, int64_t ldx, void* stream) {
    Residual res;
    res.R = R; res.ldr = ldr; res.Hout = Hout; res.ldo = ldo;
    return rmsnorm_only_impl(H, M, K, ldh, gamma, eps, X, ldx, stream, &res);
}

static osc_status rmsnorm_quantize_impl(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma,
                                        float eps, void* xq, void* sfa, void* xo, cudaStream_t st,
                                        const Residual* res = nullptr) {
    if (w->K > 8192) return fail(OSC_ERR_SHAPE, "K = %d: the fused RMSNorm stages a row in shared memory, K <= 8192", w->K);
    if (M == 0) return OSC_OK;
    if (!gamma || !aligned16(gamma)) return fail(OSC_ERR_ALIGN, "gamma must be non-null and 16-byte aligned");
    if (!xq || !sfa || (w->Kop > 0 && !xo)) return fail(OSC_ERR_INVALID_ARG, "null output pointer");
    if (!aligned16(xq) || !aligned16(sfa) || !aligned16(xo)) return fail(OSC_ERR_ALIGN, "outputs must be 16-byte aligned");
    if (res) {
        if (osc_status s = check_residual(*res, w->K)) return s;
    }
    const Residual none;
    const Residual& rs = res ? *res : none;
    cudaError_t e = launch_rmsnorm_quant(true, H, ldh, M, w->K, gamma, eps, nullptr, 0, w->idx_o, xq, sfa,
                                         w->Kop ? xo : nullptr, w->Ko, w->Kop, st, rs.R, rs.ldr, rs.Hout, rs.ldo);
    if (e != cudaSuccess) return cuda_fail(e, "rmsnorm_quant_kernel");
    return OSC_OK;
}

osc_status osc_rmsnorm_quantize_extract(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma,
                                        float eps, void* xq, void* sfa, void* xo, void* stream) {
    if (osc_status s = check_act(w, H, M, ldh)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_rmsnorm_linear_grouped_gather");
    return rmsnorm_quantize_impl(w, H, M, ldh, gamma, eps, xq, sfa, xo, static_cast<cudaStream_t>(stream));
}

osc_status osc_add_rmsnorm_quantize_extract(const osc_weights* w, const void* H, const void* R, int M, int64_t ldh,
                                            int64_t ldr, const void* gamma, float eps, void* Hout, int64_t ldo, void* xq,
                                            void* sfa, void* xo, void* stream) {
    if (osc_status s = check_act(w, H, M, ldh)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_rmsnorm_linear_grouped_gather");
    Residual res;
    res.R = R; res.ldr = ldr; res.Hout = Hout; res.ldo = ldo;
    return rmsnorm_quantize_impl(w, H, M, ldh, gamma, eps, xq, sfa, xo, static_cast<cudaStream_t>(stream), &res);
}

static osc_status rmsnorm_linear_impl(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma, float eps,
                                      void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream,
                                      const Residual* res) {
    if (osc_status s = check_act(w, H, M, ldh)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_rmsnorm_linear_grouped_gather");
    if (M == 0) return OSC_OK;
    osc_act_sizes_t sz;
    osc_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (osc_status s = rmsnorm_quantize_impl(w, H, M, ldh, gamma, eps, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, st, res))
        return s;
    return gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M, Y, ldy, nullptr, 0, nullptr, 0, st);
}

osc_status osc_rmsnorm_linear(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma, float eps,
                              void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    return rmsnorm_linear_impl(w, H, M, ldh, gamma, eps, Y, ldy, workspace, workspace_bytes, stream, nullptr);
}
osc_status osc_add_rmsnorm_linear(const osc_weights* w, const void* H, const void* R, int M, int64_t ldh, int64_t ldr,
                                  const void* gamma, float eps, void* Hout, int64_t ldo, void* Y, int64_t ldy,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    Residual res;
    res.R = R; res.ldr = ldr; res.Hout = Hout; res.ldo = ldo;
    return rmsnorm_linear_impl(w, H, M, ldh, gamma, eps, Y, ldy, workspace, workspace_bytes, stream, &res);
}

// ---- osc_linear on a gate|up handle with the activation in the epilogue: H = silu(gate) * up, [M, N/2]
// Problems of more than kSwigluFusedMinRows rows run on the pair kernel's gate|up form; smaller ones take the plain
// GEMM of the library's routing into a scratch Y behind the quantizer's buffers, then the stand-alone activation.
constexpr int kSwigluFusedMinRows = 256;
static bool swiglu_fused(const osc_weights* w, int M) {
    static const int mode = [] { const char* e = getenv("OSC_SWIGLU_FUSED"); return e ? atoi(e) : 1; }();
    if (mode == 0 || (w->N / 2) % 8) return false;
    return w->grouped ? use_pair_kernel(true, M, w->E) : M > kSwigluFusedMinRows;   // grouped: experts of 96 rows and more on average
}

osc_status osc_linear_swiglu_workspace_bytes(const osc_weights* w, int M, size_t* bytes) {
    if (!w || !bytes) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (!w->gate_up) return fail(OSC_ERR_INVALID_ARG, "not a gate|up handle: use osc_prepare_weights_gate_up");
    osc_act_sizes_t sz;
    if (osc_status s = osc_act_sizes(w, M, &sz)) return s;
    *bytes = sz.workspace_bytes + (swiglu_fused(w, M) ? 0 : align256((size_t)M * w->N * 2));
    return OSC_OK;
}

// The dual-path GEMM of a gate|up handle with the activation applied to its output: in the epilogue of the pair kernel's
// gate|up form where that runs, else the plain GEMM into `scratch_y` [M, N] and the stand-alone activation.
static osc_status gemm_swiglu_impl(const osc_weights* w, uint8_t* xq, uint8_t* sfa, uint8_t* xo, int M, void* H, int64_t ldh,
                                   const int32_t* sched, int max_tiles, const int32_t* sched2, int max_tiles2, uint8_t* scratch_y,
                                   cudaStream_t st) {
    const int I = w->N / 2;
    if (!swiglu_fused(w, M)) {
        if (osc_status s = gemm_impl(w, xq, sfa, xo, M, scratch_y, w->N, sched, max_tiles, sched2, max_tiles2, st)) return s;
        cudaError_t e = launch_swiglu_fp8(false, scratch_y, w->N, M, I, H, ldh, nullptr, nullptr, st);
        if (e != cudaSuccess) return cuda_fail(e, "swiglu_fp8_kernel(activation only)");
        return OSC_OK;
    }
    GemmArgs a;
    memset(&a, 0, sizeof a);
    if (osc_status s = make_tmap(&a.tm_a, xq, false, M, w->K / 2, w->K / 2, 128)) return s;
    if (w->Kop > 0) {
        if (osc_status s = make_tmap(&a.tm_ao, xo, true, M, (uint64_t)w->Kop * 2, (uint64_t)w->Kop * 2, 128)) return s;
    }
    a.tm_b = w->tm_b2[2];
    a.tm_bo = w->tm_bo2[2];
    a.tm_sfw = w->tm_sfw_gu;
    const uint64_t sf_row_blocks = w->grouped ? (uint64_t)max_tiles : (uint64_t)((M + 127) / 128);
    if (osc_status s = make_tmap_sf(&a.tm_sfa, sfa, sf_row_blocks * (w->K / 128))) return s;
    // H as the store target: boxes of 32 columns x 16 rows, 64-byte swizzle (a staged row is 64 bytes)
    if (osc_status s = encode_2d(&a.tm_y16, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, H, (uint64_t)I, (uint64_t)M, (uint64_t)ldh * 2, 32, 16,
                                 CU_TENSOR_MAP_SWIZZLE_64B, "H")) return s;
    a.tm_y = a.tm_y16;
    a.sfa = sfa;
    a.sfw = w->sfw;
    a.Y = static_cast<uint16_t*>(H);
    a.ldy = ldh;
    a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
    a.num_sms = w->num_sms;
    a.sched = sched; a.max_tiles = max_tiles;
    a.sched2 = sched2; a.max_tiles2 = max_tiles2;
    cudaError_t e = launch_gemm_dual_pair_swiglu(a, st);
    if (e != cudaSuccess) return cuda_fail(e, "gemm_pair_kernel(gate|up, swiglu)");
    return OSC_OK;
}

static osc_status check_h(const osc_weights* w, const void* H, int64_t ldh) {
    const int I = w->N / 2;
    if (!H) return fail(OSC_ERR_INVALID_ARG, "H is null");
    if (ldh < I) return fail(OSC_ERR_SHAPE, "ldh = %lld < I = %d", (long long)ldh, I);
    if (ldh % 8 || !aligned16(H)) return fail(OSC_ERR_ALIGN, "H must be 16-byte aligned and ldh a multiple of 8");
    return OSC_OK;
}

static osc_status linear_swiglu_impl(const osc_weights* w, const void* X, int M, int64_t ldx, const void* gamma, float eps,
                                     void* H, int64_t ldh, void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx)) return s;
    if (!w->gate_up) return fail(OSC_ERR_INVALID_ARG, "not a gate|up handle: use osc_prepare_weights_gate_up");
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_linear_swiglu_grouped");
    if (M == 0) return OSC_OK;
    osc_act_sizes_t sz;
    osc_act_sizes(w, M, &sz);
    size_t need = 0;
    osc_linear_swiglu_workspace_bytes(w, M, &need);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < need) return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    if (osc_status s = check_h(w, H, ldh)) return s;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *xq = ws + sz.xq_offset, *sfa = ws + sz.sfa_offset, *xo = ws + sz.xo_offset;
    if (gamma) {
        if (osc_status s = rmsnorm_quantize_impl(w, X, M, ldx, gamma, eps, xq, sfa, xo, st)) return s;
    } else {
        if (osc_status s = quantize_impl(w, X, M, ldx, xq, sfa, xo, nullptr, 0, st)) return s;
    }
    return gemm_swiglu_impl(w, xq, sfa, xo, M, H, ldh, nullptr, 0, nullptr, 0, ws + sz.workspace_bytes, st);
}

osc_status osc_linear_swiglu(const osc_weights* w, const void* X, int M, int64_t ldx, void* H, int64_t ldh, void* workspace,
                             size_t workspace_bytes, void* stream) {
    return linear_swiglu_impl(w, X, M, ldx, nullptr, 0.0f, H, ldh, workspace, workspace_bytes, stream);
}
osc_status osc_rmsnorm_linear_swiglu(const osc_weights* w, const void* Hin, int M, int64_t ldh_in, const void* gamma, float eps,
                                     void* H, int64_t ldh, void* workspace, size_t workspace_bytes, void* stream) {
    if (!gamma) return fail(OSC_ERR_INVALID_ARG, "gamma is null");
    return linear_swiglu_impl(w, Hin, M, ldh_in, gamma, eps, H, ldh, workspace, workspace_bytes, stream);
}

osc_status osc_linear_grouped(const osc_weights* w, const void* X_perm, const int32_t* off, int M_total, int64_t ldx,
                              void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X_perm, M_total, ldx)) return s;
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_linear");
    if (M_total == 0) return OSC_OK;
    if (!off) return fail(OSC_ERR_INVALID_ARG, "off is null");
    osc_act_sizes_t sz;
    osc_act_sizes(w, M_total, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int max_tiles = M_total / 128 + w->E;
    const int max_tiles2 = max_tiles256(M_total, w->E);
    int32_t* sched = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
    int32_t* sched2 = use_pair_kernel(true, M_total, w->E) ? sched + sched_ints(max_tiles) : nullptr;
    cudaError_t e = launch_build_sched(off, w->E, sched, max_tiles, sched2, max_tiles2, st);
    if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
    if (osc_status s = quantize_impl(w, X_perm, M_total, ldx, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset,
                                     sched, max_tiles, st)) return s;
    return gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M_total, Y, ldy, sched, max_tiles,
                     sched2, max_tiles2, st);
}

// ---- grouped linear with the dispatch fused behind the quantizer: tokens quantized once, quantized rows gathered
struct GatherLayout {
    size_t xq_u, sf_u, xo_u, total;   // offsets of the unique tokens' buffers behind the grouped workspace, and the total
};
static GatherLayout gather_layout(const osc_weights* w, int T, const osc_act_sizes_t& sz) {
    GatherLayout g;
    g.xq_u = sz.workspace_bytes;
    g.sf_u = g.xq_u + align256((size_t)T * (w->K / 2));
    g.xo_u = g.sf_u + align256((size_t)((T + 127) / 128) * (w->K / 128) * 512);
    g.total = g.xo_u + align256((size_t)T * w->Kop * 2);
    return g;
}

osc_status osc_gather_workspace_bytes(const osc_weights* w, int T, int M_total, size_t* bytes) {
    if (!w || !bytes) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights have no dispatch");
    if (T < 0 || M_total < 0) return fail(OSC_ERR_INVALID_ARG, "negative size");
    osc_act_sizes_t sz;
    if (osc_status s = osc_act_sizes(w, M_total, &sz)) return s;
    *bytes = gather_layout(w, T, sz).total;
    return OSC_OK;
}

// gamma == nullptr: X holds the activations; else X is the residual stream and the RMSNorm runs inside the quantizer
static osc_status grouped_gather_impl(const osc_weights* w, const void* X, int T, int64_t ldx, const void* gamma, float eps,
                                      const int32_t* row_token, const int32_t* off, int M_total, void* Y, int64_t ldy,
                                      void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, T, ldx)) return s;
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_linear");
    if (M_total < 0) return fail(OSC_ERR_INVALID_ARG, "M_total = %d is negative", M_total);
    if (M_total == 0) return OSC_OK;
    if (T == 0) return fail(OSC_ERR_INVALID_ARG, "rows to dispatch but no tokens");
    if (!off || !row_token) return fail(OSC_ERR_INVALID_ARG, "off / row_token is null");
    osc_act_sizes_t sz;
    osc_act_sizes(w, M_total, &sz);
    const GatherLayout g = gather_layout(w, T, sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < g.total)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, g.total);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int max_tiles = M_total / 128 + w->E;
    const int max_tiles2 = max_tiles256(M_total, w->E);
    int32_t* sched = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
    int32_t* sched2 = use_pair_kernel(true, M_total, w->E) ? sched + sched_ints(max_tiles) : nullptr;
    cudaError_t e = launch_build_sched(off, w->E, sched, max_tiles, sched2, max_tiles2, st);
    if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
    // Algorithm 2 once per token (it does not depend on the expert), as a dense problem of T rows
    if (gamma) {
        if (osc_status s = rmsnorm_quantize_impl(w, X, T, ldx, gamma, eps, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, st)) return s;
    } else {
        if (osc_status s = quantize_impl(w, X, T, ldx, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, nullptr, 0, st)) return s;
    }
    e = launch_gather_quantized(row_token, T, w->K, w->Kop, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, ws + sz.xq_offset,
                                ws + sz.sfa_offset, ws + sz.xo_offset, sched, max_tiles, st);
    if (e != cudaSuccess) return cuda_fail(e, "gather_quantized_kernel");
    return gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M_total, Y, ldy, sched, max_tiles,
                     sched2, max_tiles2, st);
}

osc_status osc_linear_grouped_gather(const osc_weights* w, const void* X, int T, int64_t ldx, const int32_t* row_token,
                                     const int32_t* off, int M_total, void* Y, int64_t ldy, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    return grouped_gather_impl(w, X, T, ldx, nullptr, 0.0f, row_token, off, M_total, Y, ldy, workspace, workspace_bytes, stream);
}

osc_status osc_rmsnorm_linear_grouped_gather(const osc_weights* w, const void* H, int T, int64_t ldh, const void* gamma,
                                             float eps, const int32_t* row_token, const int32_t* off, int M_total, void* Y,
                                             int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (!gamma) return fail(OSC_ERR_INVALID_ARG, "gamma is null");
    return grouped_gather_impl(w, H, T, ldh, gamma, eps, row_token, off, M_total, Y, ldy, workspace, workspace_bytes, stream);
}

// ---- grouped (MoE) gate|up projection with the SwiGLU in the epilogue
osc_status osc_linear_swiglu_grouped(const osc_weights* w, const void* X_perm, const int32_t* off, int M_total, int64_t ldx,
                                     void* H, int64_t ldh, void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X_perm, M_total, ldx)) return s;
    if (!w->gate_up) return fail(OSC_ERR_INVALID_ARG, "not a gate|up handle: use osc_prepare_weights_gate_up_grouped");
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_linear_swiglu");
    if (M_total == 0) return OSC_OK;
    if (!off) return fail(OSC_ERR_INVALID_ARG, "off is null");
    osc_act_sizes_t sz;
    osc_act_sizes(w, M_total, &sz);
    size_t need = 0;
    osc_linear_swiglu_workspace_bytes(w, M_total, &need);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < need) return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    if (osc_status s = check_h(w, H, ldh)) return s;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int max_tiles = M_total / 128 + w->E;
    const int max_tiles2 = max_tiles256(M_total, w->E);
    int32_t* sched = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
    int32_t* sched2 = use_pair_kernel(true, M_total, w->E) ? sched + sched_ints(max_tiles) : nullptr;
    cudaError_t e = launch_build_sched(off, w->E, sched, max_tiles, sched2, max_tiles2, st);
    if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
    uint8_t *xq = ws + sz.xq_offset, *sfa = ws + sz.sfa_offset, *xo = ws + sz.xo_offset;
    if (osc_status s = quantize_impl(w, X_perm, M_total, ldx, xq, sfa, xo, sched, max_tiles, st)) return s;
    return gemm_swiglu_impl(w, xq, sfa, xo, M_total, H, ldh, sched, max_tiles, sched2, max_tiles2, ws + sz.workspace_bytes, st);
}

// The same with the dispatch fused behind the quantizer (tokens quantized once, optionally behind an RMSNorm, their
// quantized rows gathered): workspace = the gathered call's buffers, then the scratch [M_total, 2I] if the fused form
// does not run.
osc_status osc_swiglu_gather_workspace_bytes(const osc_weights* w, int T, int M_total, size_t* bytes) {
    if (!w || !bytes) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (!w->gate_up) return fail(OSC_ERR_INVALID_ARG, "not a gate|up handle: use osc_prepare_weights_gate_up_grouped");
    size_t g = 0;
    if (osc_status s = osc_gather_workspace_bytes(w, T, M_total, &g)) return s;
    *bytes = align256(g) + (swiglu_fused(w, M_total) ? 0 : align256((size_t)M_total * w->N * 2));
    return OSC_OK;
}

static osc_status swiglu_grouped_gather_impl(const osc_weights* w, const void* X, int T, int64_t ldx, const void* gamma, float eps,
                                             const int32_t* row_token, const int32_t* off, int M_total, void* H, int64_t ldh,
                                             void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, T, ldx)) return s;
    if (!w->gate_up) return fail(OSC_ERR_INVALID_ARG, "not a gate|up handle: use osc_prepare_weights_gate_up_grouped");
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights have no dispatch");
    if (M_total < 0) return fail(OSC_ERR_INVALID_ARG, "M_total = %d is negative", M_total);
    if (M_total == 0) return OSC_OK;
    if (T == 0) return fail(OSC_ERR_INVALID_ARG, "rows to dispatch but no tokens");
    if (!off || !row_token) return fail(OSC_ERR_INVALID_ARG, "off / row_token is null");
    osc_act_sizes_t sz;
    osc_act_sizes(w, M_total, &sz);
    const GatherLayout g = gather_layout(w, T, sz);
    size_t need = 0;
    osc_swiglu_gather_workspace_bytes(w, T, M_total, &need);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < need) return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    if (osc_status s = check_h(w, H, ldh)) return s;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int max_tiles = M_total / 128 + w->E;
    const int max_tiles2 = max_tiles256(M_total, w->E);
    int32_t* sched = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
    int32_t* sched2 = use_pair_kernel(true, M_total, w->E) ? sched + sched_ints(max_tiles) : nullptr;
    cudaError_t e = launch_build_sched(off, w->E, sched, max_tiles, sched2, max_tiles2, st);
    if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
    if (gamma) {
        if (osc_status s = rmsnorm_quantize_impl(w, X, T, ldx, gamma, eps, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, st)) return s;
    } else {
        if (osc_status s = quantize_impl(w, X, T, ldx, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, nullptr, 0, st)) return s;
    }
    e = launch_gather_quantized(row_token, T, w->K, w->Kop, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, ws + sz.xq_offset,
                                ws + sz.sfa_offset, ws + sz.xo_offset, sched, max_tiles, st);
    if (e != cudaSuccess) return cuda_fail(e, "gather_quantized_kernel");
    return gemm_swiglu_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M_total, H, ldh, sched, max_tiles, sched2,
                            max_tiles2, ws + align256(g.total), st);
}

osc_status osc_linear_swiglu_grouped_gather(const osc_weights* w, const void* X, int T, int64_t ldx, const int32_t* row_token,
                                            const int32_t* off, int M_total, void* H, int64_t ldh, void* workspace,
                                            size_t workspace_bytes, void* stream) {
    return swiglu_grouped_gather_impl(w, X, T, ldx, nullptr, 0.0f, row_token, off, M_total, H, ldh, workspace, workspace_bytes, stream);
}
osc_status osc_rmsnorm_linear_swiglu_grouped_gather(const osc_weights* w, const void* Hin, int T, int64_t ldh_in, const void* gamma,
                                                    float eps, const int32_t* row_token, const int32_t* off, int M_total, void* H,
                                                    int64_t ldh, void* workspace, size_t workspace_bytes, void* stream) {
    if (!gamma) return fail(OSC_ERR_INVALID_ARG, "gamma is null");
    return swiglu_grouped_gather_impl(w, Hin, T, ldh_in, gamma, eps, row_token, off, M_total, H, ldh, workspace, workspace_bytes,
                                      stream);
}

// ------------------------------------------------------- offline profiling

osc_status osc_profile_scratch_bytes(int K, size_t* bytes) {
    if (!bytes) return fail(OSC_ERR_INVALID_ARG, "bytes is null");
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    *bytes = 256 + (size_t)(K / 32) * 32 * sizeof(int32_t);
    return OSC_OK;
}

osc_status osc_profile_lut(const void* X, int S, int K, int64_t ldx, float alpha, void* scratch, size_t scratch_bytes,
                           void* lut, void* n_hit, void* n_total, void* threshold_bits, void* stream) {
    if (S <= 0) return fail(OSC_ERR_INVALID_ARG, "S = %d must be positive", S);
    size_t need = 0;
    if (osc_status s = osc_profile_scratch_bytes(K, &need)) return s;
    if (!X || !scratch || !lut || !n_hit || !n_total || !threshold_bits) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldx < K) return fail(OSC_ERR_SHAPE, "ldx = %lld < K", (long long)ldx);
    if (ldx % 8 || !aligned16(X) || !aligned16(scratch) || (reinterpret_cast<uintptr_t>(n_hit) & 3) ||
        (reinterpret_cast<uintptr_t>(n_total) & 3) || (reinterpret_cast<uintptr_t>(threshold_bits) & 3))
        return fail(OSC_ERR_ALIGN, "X and scratch must be 16-byte aligned, ldx a multiple of 8, counters 4-byte aligned");
    if (scratch_bytes < need) return fail(OSC_ERR_WORKSPACE, "scratch has %zu bytes, %zu needed", scratch_bytes, need);
    if (!(alpha > 0.0f)) return fail(OSC_ERR_INVALID_ARG, "alpha must be positive");
    DeviceInfo di;
    if (osc_status s = device_info(&di)) return s;
    uint8_t* sc = static_cast<uint8_t*>(scratch);
    cudaError_t e = launch_profile(X, ldx, S, K, (double)alpha, reinterpret_cast<double*>(sc),
                                   reinterpret_cast<int32_t*>(sc + 256), static_cast<int8_t*>(lut),
                                   static_cast<int32_t*>(n_hit), static_cast<int32_t*>(n_total),
                                   static_cast<uint32_t*>(threshold_bits), di.num_sms, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "profile kernels");
    return OSC_OK;
}

// -------------------------------------------------------------- FP8 fallback

static osc_status fp8_prepare_impl(const void* W, int E, int N, int K, int64_t ldw, void* w8, void* sw, void* stream,
                                   bool grouped, osc_fp8_weights** out) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if (osc_status s = check_nk(E, N, K)) return s;
    if (!W || !w8 || !sw) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldw < K) return fail(OSC_ERR_SHAPE, "ldw = %lld < K", (long long)ldw);
    if (ldw % 8 || !aligned16(W) || !aligned16(w8) || !aligned16(sw))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldw a multiple of 8");
    DeviceInfo di;
    if (osc_status s = device_info(&di)) return s;
    cudaError_t e = launch_fp8_quant(W, ldw, E * N, K, w8, sw, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "fp8_quant_kernel(weights)");
    e = launch_prepare_fence(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "prepare_fence_kernel");
    osc_fp8_weights* w = new (std::nothrow) osc_fp8_weights();
    if (!w) return fail(OSC_ERR_INVALID_ARG, "out of host memory");
    w->E = E; w->N = N; w->K = K; w->grouped = grouped;
    w->w8 = static_cast<const uint8_t*>(w8);
    w->sw = static_cast<const float*>(sw);
    w->num_sms = di.num_sms;
    for (int v = 0; v < 4; ++v) {
        if (osc_status s = make_tmap(&w->tm_b[v], w8, false, (uint64_t)E * N, K, K, 64 * (v + 1))) { delete w; return s; }
    }
    for (int v = 0; v < 2; ++v) {
        if (osc_status s = make_tmap(&w->tm_b2[v], w8, false, (uint64_t)E * N, K, K, (v == 0 ? 192 : 256) / 2)) { delete w; return s; }
    }
    *out = w;
    return OSC_OK;
}

osc_status osc_fp8_prepare_weights(const void* W, int N, int K, int64_t ldw, void* w8, void* sw, void* stream,
                                   osc_fp8_weights** out) {
    return fp8_prepare_impl(W, 1, N, K, ldw, w8, sw, stream, false, out);
}
osc_status osc_fp8_prepare_weights_grouped(const void* W, int E, int N, int K, void* w8, void* sw, void* stream,
                                           osc_fp8_weights** out) {
    return fp8_prepare_impl(W, E, N, K, K, w8, sw, stream, true, out);
}
osc_status osc_fp8_weights_destroy(osc_fp8_weights* w) {
    delete w;
    return OSC_OK;
}

osc_status osc_fp8_act_sizes(const osc_fp8_weights* w, int M, osc_fp8_act_sizes_t* out) {
    if (!w || !out) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    const int64_t max_tiles = w->grouped ? (int64_t)M / 128 + w->E : 0;
    out->x8_bytes = (size_t)M * w->K;
    out->sx_bytes = (size_t)M * 4;
    out->sched_bytes = w->grouped ? sched_ints(max_tiles) * 4 + sched_ints(max_tiles256(M, w->E)) * 4 : 0;
    out->x8_offset = 0;
    out->sx_offset = align256(out->x8_bytes);
    out->sched_offset = out->sx_offset + align256(out->sx_bytes);
    out->workspace_bytes = out->sched_offset + align256(out->sched_bytes);
    return OSC_OK;
}

osc_status osc_fp8_quantize(const void* X, int M, int K, int64_t ldx, void* x8, void* sx, void* stream) {
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    if (M == 0) return OSC_OK;
    if (!X || !x8 || !sx) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldx < K) return fail(OSC_ERR_SHAPE, "ldx = %lld < K", (long long)ldx);
    if (ldx % 8 || !aligned16(X) || !aligned16(x8) || !aligned16(sx))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldx a multiple of 8");
    cudaError_t e = launch_fp8_quant(X, ldx, M, K, x8, sx, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "fp8_quant_kernel");
    return OSC_OK;
}

static osc_status fp8_gemm_impl(const osc_fp8_weights* w, const void* x8, const void* sx, int M, void* Y, int64_t ldy,
                                const int32_t* sched, int max_tiles, const int32_t* sched2, int max_tiles2,
                                cudaStream_t st) {
    if (M == 0) return OSC_OK;
    if (!x8 || !sx || !Y) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y) || !aligned16(x8) || !aligned16(sx))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldy a multiple of 8");
    GemmArgs a;
    memset(&a, 0, sizeof a);
    if (use_decode_kernel(w->grouped, M, w->N, w->K / 128, w->num_sms)) {
        if (osc_status s = make_tmap(&a.tm_a, x8, false, M, w->K, w->K, (uint32_t)((M + 15) / 16 * 16))) return s;
        a.tm_b = w->tm_b[1];
        a.sx = static_cast<const float*>(sx);
        a.sw = w->sw;
        a.Y = static_cast<uint16_t*>(Y);
        a.ldy = ldy;
        a.M = M; a.N = w->N; a.K = w->K; a.Kop = 0;
        a.num_sms = w->num_sms;
        const int S = gemm_decode_split(w->N, w->K / 128, w->num_sms);
        cudaError_t e = launch_gemm_fp8_decode(a, S, st);
        if (e != cudaSuccess) return cuda_fail(e, "gemm_decode_kernel(fp8)");
        return OSC_OK;
    }
    if (osc_status s = make_tmap(&a.tm_a, x8, false, M, w->K, w->K, 128)) return s;
    long single_ns = 0, pair_ns = 0;
    const int bn1 = gemm_block_n(sched ? max_tiles : (M + 127) / 128, w->N, w->num_sms, &single_ns);
    const long row_tiles2 = w->grouped ? (max_tiles2 > w->E / 2 ? max_tiles2 - w->E / 2 : 1) : (M + 255) / 256;
    const int bn2 = gemm_pair_block_n(true, false, row_tiles2, w->N, w->K / 128, w->num_sms, &pair_ns);
    a.tm_b = w->tm_b[bn1 / 64 - 1];
    a.sx = static_cast<const float*>(sx);
    a.sw = w->sw;
    a.Y = static_cast<uint16_t*>(Y);
    a.ldy = ldy;
    a.M = M; a.N = w->N; a.K = w->K; a.Kop = 0;
    a.sched = sched; a.max_tiles = max_tiles; a.num_sms = w->num_sms;
    a.sched2 = sched2; a.max_tiles2 = max_tiles2;
    cudaError_t e;
    if (use_pair_kernel(w->grouped, M, w->E, single_ns * (w->K / 128), pair_ns, single_ns <= 470)) {
        const int bn = bn2;
        a.tm_b = w->tm_b2[bn == 256];
        if (osc_status s = make_tmap(&a.tm_y, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 32)) return s;
        if (osc_status s = make_tmap(&a.tm_y16, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 16)) return s;
        e = launch_gemm_fp8_pair(a, bn, st);
    } else {
        e = launch_gemm_fp8(a, bn1, st);
    }
    if (e != cudaSuccess) return cuda_fail(e, "gemm_kernel(fp8)");
    return OSC_OK;
}

osc_status osc_fp8_gemm(const osc_fp8_weights* w, const void* x8, const void* sx, int M, void* Y, int64_t ldy,
                        void* stream) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_fp8_linear_grouped");
    return fp8_gemm_impl(w, x8, sx, M, Y, ldy, nullptr, 0, nullptr, 0, static_cast<cudaStream_t>(stream));
}

static osc_status check_swiglu(const void* GU, int M, int I, int64_t ldg);

// swiglu: X is the gate|up matrix [M, 2K] and the quantizer computes the activation on the way in
static osc_status fp8_linear_impl(const osc_fp8_weights* w, const void* X, const int32_t* off, int M, int64_t ldx,
                                  void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream,
                                  bool swiglu = false) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (swiglu) {
        if (osc_status s = check_swiglu(X, M, w->K, ldx)) return s;
    }
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (M == 0) return OSC_OK;
    if (w->grouped && !off) return fail(OSC_ERR_INVALID_ARG, "off is null");
    if (!swiglu) {   // what osc_fp8_quantize would refuse, refused before the schedule builder is launched
        if (!X) return fail(OSC_ERR_INVALID_ARG, "X is null");
        if (ldx < w->K) return fail(OSC_ERR_SHAPE, "ldx = %lld < K", (long long)ldx);
        if (ldx % 8 || !aligned16(X)) return fail(OSC_ERR_ALIGN, "X must be 16-byte aligned and ldx a multiple of 8");
    }
    osc_fp8_act_sizes_t sz;
    osc_fp8_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int32_t *sched = nullptr, *sched2 = nullptr;
    int max_tiles = 0, max_tiles2 = 0;
    if (w->grouped) {
        // only the schedule of the GEMM kernel that will run (the FP8 quantizer needs none)
        max_tiles = M / 128 + w->E;
        max_tiles2 = max_tiles256(M, w->E);
        int32_t* s = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
        const bool pair = use_pair_kernel(true, M, w->E);
        cudaError_t e = launch_build_sched(off, w->E, pair ? nullptr : s, max_tiles, pair ? s + sched_ints(max_tiles) : nullptr,
                                           max_tiles2, st);
        if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
        if (pair) sched2 = s + sched_ints(max_tiles); else sched = s;
    }
    if (swiglu) {
        if (osc_status s = osc_swiglu_fp8_quantize(X, M, w->K, ldx, ws + sz.x8_offset, ws + sz.sx_offset, stream)) return s;
    } else {
        if (osc_status s = osc_fp8_quantize(X, M, w->K, ldx, ws + sz.x8_offset, ws + sz.sx_offset, stream)) return s;
    }
    return fp8_gemm_impl(w, ws + sz.x8_offset, ws + sz.sx_offset, M, Y, ldy, sched, max_tiles, sched2, max_tiles2, st);
}

osc_status osc_fp8_linear(const osc_fp8_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (w && w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_fp8_linear_grouped");
    return fp8_linear_impl(w, X, nullptr, M, ldx, Y, ldy, workspace, workspace_bytes, stream);
}
osc_status osc_fp8_linear_grouped(const osc_fp8_weights* w, const void* X_perm, const int32_t* off, int M_total,
                                  int64_t ldx, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                  void* stream) {
    if (w && !w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_fp8_linear");
    return fp8_linear_impl(w, X_perm, off, M_total, ldx, Y, ldy, workspace, workspace_bytes, stream);
}

// ---- SwiGLU fused in front of the per-token FP8 quantizer
static osc_status check_swiglu(const void* GU, int M, int I, int64_t ldg) {
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (I <= 0 || I % 128) return fail(OSC_ERR_SHAPE, "I = %d must be a positive multiple of 128", I);
    if (I > 16384) return fail(OSC_ERR_SHAPE, "I = %d: the fused SwiGLU holds a row in registers, I <= 16384", I);
    if (M > 0 && !GU) return fail(OSC_ERR_INVALID_ARG, "GU is null");
    if (ldg < 2 * (int64_t)I) return fail(OSC_ERR_SHAPE, "ldg = %lld < 2 I = %d", (long long)ldg, 2 * I);
    if (ldg % 8 || !aligned16(GU)) return fail(OSC_ERR_ALIGN, "GU must be 16-byte aligned and ldg a multiple of 8");
    return OSC_OK;
}

osc_status osc_swiglu(const void* GU, int M, int I, int64_t ldg, void* H, int64_t ldh, void* stream) {
    if (osc_status s = check_swiglu(GU, M, I, ldg)) return s;
    if (M == 0) return OSC_OK;
    if (!H) return fail(OSC_ERR_INVALID_ARG, "H is null");
    if (ldh < I) return fail(OSC_ERR_SHAPE, "ldh = %lld < I = %d", (long long)ldh, I);
    if (ldh % 8 || !aligned16(H)) return fail(OSC_ERR_ALIGN, "H must be 16-byte aligned and ldh a multiple of 8");
    cudaError_t e = launch_swiglu_fp8(false, GU, ldg, M, I, H, ldh, nullptr, nullptr, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "swiglu_fp8_kernel(activation only)");
    return OSC_OK;
}

osc_status osc_swiglu_fp8_quantize(const void* GU, int M, int I, int64_t ldg, void* x8, void* sx, void* stream) {
    if (osc_status s = check_swiglu(GU, M, I, ldg)) return s;
    if (M == 0) return OSC_OK;
    if (!x8 || !sx) return fail(OSC_ERR_INVALID_ARG, "null output pointer");
    if (!aligned16(x8) || !aligned16(sx)) return fail(OSC_ERR_ALIGN, "outputs must be 16-byte aligned");
    cudaError_t e = launch_swiglu_fp8(true, GU, ldg, M, I, nullptr, 0, x8, sx, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "swiglu_fp8_kernel");
    return OSC_OK;
}

osc_status osc_swiglu_fp8_linear(const osc_fp8_weights* w, const void* GU, int M, int64_t ldg, void* Y, int64_t ldy,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    if (w && w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_swiglu_fp8_linear_grouped");
    return fp8_linear_impl(w, GU, nullptr, M, ldg, Y, ldy, workspace, workspace_bytes, stream, true);
}
osc_status osc_swiglu_fp8_linear_grouped(const osc_fp8_weights* w, const void* GU_perm, const int32_t* off, int M_total,
                                         int64_t ldg, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                         void* stream) {
    if (w && !w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_swiglu_fp8_linear");
    return fp8_linear_impl(w, GU_perm, off, M_total, ldg, Y, ldy, workspace, workspace_bytes, stream, true);
}

// ------------------------------------------------- MXFP8 form of the fallback

osc_status osc_mxfp8_weight_sizes(int E, int N, int K, osc_mxfp8_weight_sizes_t* out) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    if (osc_status s = check_nk(E, N, K)) return s;
    out->w8_bytes = (size_t)E * N * K;
    out->sfw_bytes = (size_t)E * sf_bytes(N, K);
    return OSC_OK;
}

static osc_status mxfp8_quantize_impl(const void* X, int M, int K, int64_t ldx, void* x8, void* sfa,
                                      const int32_t* sched, int max_tiles, void* stream) {
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    if (M == 0) return OSC_OK;
    if (!X || !x8 || !sfa) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldx < K) return fail(OSC_ERR_SHAPE, "ldx = %lld < K", (long long)ldx);
    if (ldx % 8 || !aligned16(X) || !aligned16(x8) || !aligned16(sfa))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldx a multiple of 8");
    cudaError_t e = launch_mxfp8_quant(X, ldx, M, K, x8, sfa, sched, max_tiles, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "mxfp8_quant_kernel");
    return OSC_OK;
}

osc_status osc_mxfp8_quantize(const void* X, int M, int K, int64_t ldx, void* x8, void* sfa, void* stream) {
    return mxfp8_quantize_impl(X, M, K, ldx, x8, sfa, nullptr, 0, stream);
}

static osc_status mxfp8_prepare_impl(const void* W, int E, int N, int K, int64_t ldw, void* w8, void* sfw, void* stream,
                                     bool grouped, osc_mxfp8_weights** out) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if (osc_status s = check_nk(E, N, K)) return s;
    DeviceInfo di;
    if (osc_status s = device_info(&di)) return s;
    // expert by expert: every expert's scales start on a 128-row block of their own
    for (int ex = 0; ex < E; ++ex) {
        if (osc_status s = mxfp8_quantize_impl(static_cast<const uint16_t*>(W) + (size_t)ex * N * ldw, N, K, ldw,
                                               static_cast<uint8_t*>(w8) + (size_t)ex * N * K,
                                               static_cast<uint8_t*>(sfw) + (size_t)ex * sf_bytes(N, K), nullptr, 0, stream))
            return s;
    }
    if (cudaError_t e = launch_prepare_fence(static_cast<cudaStream_t>(stream))) return cuda_fail(e, "prepare_fence_kernel");
    osc_mxfp8_weights* w = new (std::nothrow) osc_mxfp8_weights();
    if (!w) return fail(OSC_ERR_INVALID_ARG, "out of host memory");
    w->E = E; w->N = N; w->K = K; w->grouped = grouped;
    w->w8 = static_cast<const uint8_t*>(w8);
    w->sfw = static_cast<const uint8_t*>(sfw);
    w->num_sms = di.num_sms;
    osc_status s = OSC_OK;
    for (int v = 0; v < 2 && s == OSC_OK; ++v)
        s = make_tmap(&w->tm_b2[v], w8, false, (uint64_t)E * N, K, K, (v == 0 ? 192 : 256) / 2);
    if (s == OSC_OK) s = make_tmap(&w->tm_b128, w8, false, (uint64_t)E * N, K, K, 128);
    for (int v = 0; v < 4 && s == OSC_OK; ++v) s = make_tmap(&w->tm_b1[v], w8, false, (uint64_t)E * N, K, K, 64 * (v + 1));
    if (s == OSC_OK) s = make_tmap_sf(&w->tm_sfw, sfw, (uint64_t)E * sf_bytes(N, K) / 512, 1);
    if (s != OSC_OK) { delete w; return s; }
    *out = w;
    return OSC_OK;
}
osc_status osc_mxfp8_prepare_weights(const void* W, int N, int K, int64_t ldw, void* w8, void* sfw, void* stream,
                                     osc_mxfp8_weights** out) {
    return mxfp8_prepare_impl(W, 1, N, K, ldw, w8, sfw, stream, false, out);
}
osc_status osc_mxfp8_prepare_weights_grouped(const void* W, int E, int N, int K, void* w8, void* sfw, void* stream,
                                             osc_mxfp8_weights** out) {
    return mxfp8_prepare_impl(W, E, N, K, K, w8, sfw, stream, true, out);
}
osc_status osc_mxfp8_weights_destroy(osc_mxfp8_weights* w) {
    delete w;
    return OSC_OK;
}

osc_status osc_mxfp8_act_sizes(const osc_mxfp8_weights* w, int M, osc_mxfp8_act_sizes_t* out) {
    if (!w || !out) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    const int64_t max_tiles = w->grouped ? (int64_t)M / 128 + w->E : ((int64_t)M + 127) / 128;
    out->x8_bytes = (size_t)M * w->K;
    out->sfa_bytes = (size_t)max_tiles * (w->K / 128) * 512;
    out->sched_bytes = w->grouped ? sched_ints(max_tiles) * 4 + sched_ints(max_tiles256(M, w->E)) * 4 : 0;
    out->x8_offset = 0;
    out->sfa_offset = align256(out->x8_bytes);
    out->sched_offset = out->sfa_offset + align256(out->sfa_bytes);
    out->workspace_bytes = out->sched_offset + align256(out->sched_bytes);
    return OSC_OK;
}

static osc_status mxfp8_gemm_impl(const osc_mxfp8_weights* w, const void* x8, const void* sfa, int M, void* Y,
                                  int64_t ldy, const int32_t* sched, const int32_t* sched2, int max_tiles, int max_tiles2,
                                  void* stream) {
    if (M == 0) return OSC_OK;
    if (!x8 || !sfa || !Y) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y) || !aligned16(x8) || !aligned16(sfa))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldy a multiple of 8");
    GemmArgs a;
    memset(&a, 0, sizeof a);
    if (use_decode_kernel(w->grouped, M, w->N, w->K / 128, w->num_sms)) {
        if (osc_status s = make_tmap(&a.tm_a, x8, false, M, w->K, w->K, (uint32_t)((M + 15) / 16 * 16))) return s;
        a.tm_b = w->tm_b128;
        a.sfa = static_cast<const uint8_t*>(sfa);
        a.sfw = w->sfw;
        a.Y = static_cast<uint16_t*>(Y);
        a.ldy = ldy;
        a.M = M; a.N = w->N; a.K = w->K; a.Kop = 0;
        a.num_sms = w->num_sms;
        const int S = gemm_decode_split(w->N, w->K / 128, w->num_sms);
        cudaError_t e = launch_gemm_mxf8_decode(a, S, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "gemm_decode_kernel(mxfp8)");
        return OSC_OK;
    }
    if (osc_status s = make_tmap(&a.tm_a, x8, false, M, w->K, w->K, 128)) return s;
    // grouped problems with large experts run on the CTA-pair kernel (256-row tiles; rows past the end are zero-filled by
    // the loads or belong to the next expert, and are never stored), those with small experts on 128-row tiles; dense
    // ones on whichever kernel its cost model puts ahead
    const long row_tiles = w->grouped ? (max_tiles2 > w->E / 2 ? max_tiles2 - w->E / 2 : 1) : (M + 255) / 256;
    long single_ns = 0, pair_ns = 0;
    const int bn1 = gemm_block_n(w->grouped ? max_tiles : (M + 127) / 128, w->N, w->num_sms, &single_ns);
    const int bn = gemm_pair_block_n(false, false, row_tiles, w->N, w->K / 128, w->num_sms, &pair_ns);
    if (!use_pair_kernel(w->grouped, M, w->E, single_ns * (w->K / 128), pair_ns, single_ns <= 470)) {
        a.tm_b = w->tm_b1[bn1 / 64 - 1];
        a.sched = sched; a.max_tiles = max_tiles;
        a.sfa = static_cast<const uint8_t*>(sfa);
        a.sfw = w->sfw;
        a.Y = static_cast<uint16_t*>(Y);
        a.ldy = ldy;
        a.M = M; a.N = w->N; a.K = w->K; a.Kop = 0;
        a.num_sms = w->num_sms;
        cudaError_t e1 = launch_gemm_mxf8(a, bn1, static_cast<cudaStream_t>(stream));
        if (e1 != cudaSuccess) return cuda_fail(e1, "gemm_kernel(mxfp8)");
        return OSC_OK;
    }
    a.tm_b = w->tm_b2[bn == 256];
    a.tm_sfw = w->tm_sfw;
    const uint64_t sf_row_blocks = w->grouped ? (uint64_t)max_tiles : (uint64_t)((M + 127) / 128);
    if (osc_status s = make_tmap_sf(&a.tm_sfa, sfa, sf_row_blocks * (w->K / 128), 1)) return s;
    if (osc_status s = make_tmap(&a.tm_y, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 32)) return s;
    if (osc_status s = make_tmap(&a.tm_y16, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 16)) return s;
    a.sfa = static_cast<const uint8_t*>(sfa);
    a.sfw = w->sfw;
    a.Y = static_cast<uint16_t*>(Y);
    a.ldy = ldy;
    a.M = M; a.N = w->N; a.K = w->K; a.Kop = 0;
    a.num_sms = w->num_sms;
    a.sched2 = sched2; a.max_tiles2 = max_tiles2;
    cudaError_t e = launch_gemm_mxf8_pair(a, bn, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "gemm_pair_kernel(mxfp8)");
    return OSC_OK;
}

osc_status osc_mxfp8_gemm(const osc_mxfp8_weights* w, const void* x8, const void* sfa, int M, void* Y, int64_t ldy,
                          void* stream) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_mxfp8_linear_grouped");
    return mxfp8_gemm_impl(w, x8, sfa, M, Y, ldy, nullptr, nullptr, 0, 0, stream);
}

static osc_status mxfp8_linear_impl(const osc_mxfp8_weights* w, const void* X, const int32_t* off, int M, int64_t ldx,
                                    void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (M == 0) return OSC_OK;
    if (w->grouped && !off) return fail(OSC_ERR_INVALID_ARG, "off is null");
    osc_mxfp8_act_sizes_t sz;
    osc_mxfp8_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int32_t *sched = nullptr, *sched2 = nullptr;
    int max_tiles = 0, max_tiles2 = 0;
    if (w->grouped) {
        max_tiles = M / 128 + w->E;
        max_tiles2 = max_tiles256(M, w->E);
        int32_t* s1 = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
        int32_t* s2 = s1 + sched_ints(max_tiles);
        cudaError_t e = launch_build_sched(off, w->E, s1, max_tiles, s2, max_tiles2, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
        sched = s1;
        sched2 = s2;
    }
    if (osc_status s = mxfp8_quantize_impl(X, M, w->K, ldx, ws + sz.x8_offset, ws + sz.sfa_offset, sched, max_tiles, stream))
        return s;
    return mxfp8_gemm_impl(w, ws + sz.x8_offset, ws + sz.sfa_offset, M, Y, ldy, sched, sched2, max_tiles, max_tiles2, stream);
}

osc_status osc_mxfp8_linear(const osc_mxfp8_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* stream) {
    if (w && w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_mxfp8_linear_grouped");
    return mxfp8_linear_impl(w, X, nullptr, M, ldx, Y, ldy, workspace, workspace_bytes, stream);
}
osc_status osc_mxfp8_linear_grouped(const osc_mxfp8_weights* w, const void* X_perm, const int32_t* off, int M_total,
                                    int64_t ldx, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                    void* stream) {
    if (w && !w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_mxfp8_linear");
    return mxfp8_linear_impl(w, X_perm, off, M_total, ldx, Y, ldy, workspace, workspace_bytes, stream);
}

// ------------------------------- dynamic-protection control group (Section 4.2)

osc_status osc_dyn_weight_sizes(int N, int K, osc_weight_sizes_t* out) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    if (osc_status s = check_nk(1, N, K)) return s;
    out->K_o = K;
    out->K_o_pad = K;
    out->wq_bytes = (size_t)N * (K / 2);
    out->sfw_bytes = sf_bytes(N, K);
    out->wo_bytes = (size_t)N * K * 2;
    out->meta_bytes = meta_table_bytes(K, 0) + tiled_sf_bytes(N, K);
    return OSC_OK;
}

osc_status osc_dyn_prepare_weights(const void* W, int N, int K, int64_t ldw, void* wq, void* sfw, void* wo, void* meta,
                                   void* stream, osc_weights** out) {
    return prepare_impl(W, 1, N, K, ldw, nullptr, 0, wq, sfw, wo, meta, stream, false, out, true);
}

osc_status osc_dyn_act_sizes(const osc_weights* w, int M, osc_dyn_act_sizes_t* out) {
    if (!w || !out) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (!w->dynamic) return fail(OSC_ERR_INVALID_ARG, "static-table weights: use osc_act_sizes");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    out->xq_bytes = (size_t)M * (w->K / 2);
    out->sfa_bytes = sf_bytes(M, w->K);
    out->xo_bytes = (size_t)M * w->K * 2;
    out->idx_bytes = (size_t)M * (w->K / 32);
    out->val_bytes = (size_t)M * (w->K / 32) * 2;
    out->xq_offset = 0;
    out->sfa_offset = out->xq_offset + align256(out->xq_bytes);
    out->xo_offset = out->sfa_offset + align256(out->sfa_bytes);
    out->idx_offset = out->xo_offset + align256(out->xo_bytes);
    out->val_offset = out->idx_offset + align256(out->idx_bytes);
    out->workspace_bytes = out->val_offset + align256(out->val_bytes);
    return OSC_OK;
}

osc_status osc_dyn_quantize_extract(const osc_weights* w, const void* X, int M, int64_t ldx, void* xq, void* sfa,
                                    void* xo, void* idx, void* val, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx, true)) return s;
    if (M == 0) return OSC_OK;
    if (!xq || !sfa || !xo || !idx || !val) return fail(OSC_ERR_INVALID_ARG, "null output pointer");
    if (!aligned16(xq) || !aligned16(sfa) || !aligned16(xo) || !aligned16(idx) || !aligned16(val))
        return fail(OSC_ERR_ALIGN, "outputs must be 16-byte aligned");
    cudaError_t e = launch_dyn_quant_extract(X, ldx, M, w->K, xq, sfa, xo, idx, val, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "dyn_quant_extract_kernel");
    return OSC_OK;
}

osc_status osc_dyn_linear(const osc_weights* w, const void* X, int M, int64_t ldx, void* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx, true)) return s;
    if (M == 0) return OSC_OK;
    osc_dyn_act_sizes_t sz;
    osc_dyn_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (osc_status s = osc_dyn_quantize_extract(w, X, M, ldx, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset,
                                                ws + sz.idx_offset, ws + sz.val_offset, stream)) return s;
    return gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M, Y, ldy, nullptr, 0, nullptr, 0,
                     static_cast<cudaStream_t>(stream));
}

// ------------------------------------------------ NVFP4 / G = 16 variant

static size_t sf16_bytes(int64_t rows, int K) { return (size_t)((rows + 127) / 128) * (K / 64) * 512; }

// table for 16-channel groups [K/16][C] (entries -1..15) -> the 32-group form the kernels use [K/32][2C]
static osc_status widen_lut16(const int8_t* lut16, int K, int C, std::vector<int8_t>* out) {
    if (K <= 0 || K % 128) return fail(OSC_ERR_SHAPE, "K = %d must be a positive multiple of 128", K);
    if (C < 0 || C > 16) return fail(OSC_ERR_INVALID_ARG, "lut_c = %d outside 0..16", C);
    if (C > 0 && !lut16) return fail(OSC_ERR_INVALID_ARG, "lut is null");
    out->assign((size_t)(K / 32) * 2 * (C > 0 ? C : 1), -1);
    for (int g = 0; g < K / 16; ++g)
        for (int c = 0; c < C; ++c) {
            const int j = lut16[(size_t)g * C + c];
            if (j < -1 || j > 15) return fail(OSC_ERR_LUT, "table entry %d of group %d outside -1..15", j, g);
            if (j >= 0) (*out)[(size_t)(g / 2) * 2 * C + (g & 1) * C + c] = (int8_t)(j + 16 * (g & 1));
        }
    return OSC_OK;
}

osc_status osc_nvfp4_weight_sizes(int N, int K, const int8_t* lut16, int lut_c, osc_weight_sizes_t* out) {
    return osc_nvfp4_weight_sizes_grouped(1, N, K, lut16, lut_c, out);
}
osc_status osc_nvfp4_weight_sizes_grouped(int E, int N, int K, const int8_t* lut16, int lut_c, osc_weight_sizes_t* out) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    if (osc_status s = check_nk(E, N, K)) return s;
    std::vector<int8_t> lut;
    if (osc_status s = widen_lut16(lut16, K, lut_c, &lut)) return s;
    Table t;
    if (osc_status s = parse_lut(lut.data(), K, 2 * (lut_c > 0 ? lut_c : 1), &t)) return s;
    out->K_o = t.Ko;
    out->K_o_pad = t.Kop;
    out->wq_bytes = (size_t)E * N * (K / 2);
    out->sfw_bytes = (size_t)E * sf16_bytes(N, K);
    out->wo_bytes = (size_t)E * N * t.Kop * 2;
    // dense: the per-tile copy of the weight scales for 240-wide tiles (scale blocks of 64 channels: twice the MXFP4 copy)
    out->meta_bytes = meta_table_bytes(K, t.Ko) + (E == 1 ? 2 * tiled_sf_bytes(N, K) : 0);
    return OSC_OK;
}

static osc_status nvfp4_prepare_impl(const void* W, int E, int N, int K, int64_t ldw, const int8_t* lut16, int lut_c, int ew,
                                     void* wq, void* sfw, void* wo, void* meta, void* stream, osc_weights** out,
                                     bool grouped) {
    if (!out) return fail(OSC_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if (osc_status s = check_nk(E, N, K)) return s;
    if (ew < -100 || ew > 100) return fail(OSC_ERR_INVALID_ARG, "tensor exponent %d outside -100..100", ew);
    std::vector<int8_t> lut;
    if (osc_status s = widen_lut16(lut16, K, lut_c, &lut)) return s;
    Table t;
    if (osc_status s = parse_lut(lut.data(), K, 2 * (lut_c > 0 ? lut_c : 1), &t)) return s;
    if (!W || !wq || !sfw || !meta || (t.Kop > 0 && !wo)) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldw < K) return fail(OSC_ERR_SHAPE, "ldw = %lld < K", (long long)ldw);
    if (ldw % 8 || !aligned16(W) || !aligned16(wq) || !aligned16(sfw) || !aligned16(meta) || !aligned16(wo))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldw a multiple of 8");
    DeviceInfo di;
    if (osc_status s = device_info(&di)) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int Kg = K / 32;
    uint8_t* m8 = static_cast<uint8_t*>(meta);
    cudaError_t e = cudaMemcpyAsync(m8, t.mask.data(), (size_t)Kg * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(m8 + (size_t)Kg * 4, t.prefix.data(), (size_t)Kg * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && t.Ko > 0)
        e = cudaMemcpyAsync(m8 + (size_t)Kg * 8, t.idx.data(), (size_t)t.Ko * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(meta)");
    osc_weights* w = new (std::nothrow) osc_weights();
    if (!w) return fail(OSC_ERR_INVALID_ARG, "out of host memory");
    w->E = E; w->N = N; w->K = K; w->Ko = t.Ko; w->Kop = t.Kop; w->grouped = grouped; w->dynamic = false;
    w->nvfp4 = true; w->ew = ew;
    w->wq = static_cast<const uint8_t*>(wq);
    w->sfw = static_cast<const uint8_t*>(sfw);
    w->wo = static_cast<const uint16_t*>(wo);
    w->mask = reinterpret_cast<const uint32_t*>(m8);
    w->prefix = reinterpret_cast<const int32_t*>(m8 + (size_t)Kg * 4);
    w->idx_o = reinterpret_cast<const int32_t*>(m8 + (size_t)Kg * 8);
    w->num_sms = di.num_sms;
    osc_status s = OSC_OK;
    const size_t sfw_e = sf16_bytes(N, K);
    for (int x = 0; x < E && s == OSC_OK; ++x) {   // every expert on its own: its scale blocks start on a 128-row block
        CUtensorMap tm_w;
        s = make_tmap_x(&tm_w, static_cast<const uint16_t*>(W) + (size_t)x * N * ldw, N, K, ldw);
        if (s != OSC_OK) break;
        e = launch_quant_extract_nvfp4(tm_w, N, K, w->mask, w->prefix, w->idx_o, static_cast<uint8_t*>(wq) + (size_t)x * N * (K / 2),
                                       static_cast<uint8_t*>(sfw) + (size_t)x * sfw_e,
                                       t.Kop ? static_cast<uint16_t*>(wo) + (size_t)x * N * t.Kop : nullptr, t.Ko, t.Kop,
                                       di.num_sms, ew, st);
        if (e != cudaSuccess) s = cuda_fail(e, "quant_extract_kernel(nvfp4 weights)");
    }
    if (s == OSC_OK && !grouped) {   // 240-wide tiles read a per-tile copy of the weight scales (behind the table in meta)
        uint8_t* tiled = m8 + meta_table_bytes(K, t.Ko);
        e = launch_retile_sf(static_cast<const uint8_t*>(sfw), tiled, N, K, kTiledBN, st, false, 64);
        if (e != cudaSuccess) s = cuda_fail(e, "retile_sf_kernel(nvfp4)");
        if (s == OSC_OK) s = make_tmap_sf(&w->tm_sfw_tiled, tiled, (uint64_t)(2 * tiled_sf_bytes(N, K)) / 512, 4);
    }
    if (s == OSC_OK && (e = launch_prepare_fence(st)) != cudaSuccess) s = cuda_fail(e, "prepare_fence_kernel");
    for (int v = 0; v < (grouped ? 2 : 3) && s == OSC_OK; ++v) {
        const int half = (v == 0 ? 192 : v == 1 ? 256 : kTiledBN) / 2;
        s = make_tmap(&w->tm_b2[v], wq, false, (uint64_t)E * N, K / 2, K / 2, half);
        if (s == OSC_OK && t.Kop > 0)
            s = make_tmap(&w->tm_bo2[v], wo, true, (uint64_t)E * N, (uint64_t)t.Kop * 2, (uint64_t)t.Kop * 2, half);
    }
    if (s == OSC_OK) s = make_tmap_sf(&w->tm_sfw, sfw, (uint64_t)E * sfw_e / 512, 4);
    // weight tiles of the few-row kernel (128 rows) and of the 128-row-tile kernel (64, 128, 192 rows)
    for (int v = 0; v < 3 && s == OSC_OK; ++v) {
        s = make_tmap(&w->tm_b[v], wq, false, (uint64_t)E * N, K / 2, K / 2, 64 * (v + 1));
        if (s == OSC_OK && t.Kop > 0)
            s = make_tmap(&w->tm_bo[v], wo, true, (uint64_t)E * N, (uint64_t)t.Kop * 2, (uint64_t)t.Kop * 2, 64 * (v + 1));
    }
    if (s != OSC_OK) { delete w; return s; }
    *out = w;
    return OSC_OK;
}

osc_status osc_nvfp4_prepare_weights(const void* W, int N, int K, int64_t ldw, const int8_t* lut16, int lut_c, int ew,
                                     void* wq, void* sfw, void* wo, void* meta, void* stream, osc_weights** out) {
    return nvfp4_prepare_impl(W, 1, N, K, ldw, lut16, lut_c, ew, wq, sfw, wo, meta, stream, out, false);
}
osc_status osc_nvfp4_prepare_weights_grouped(const void* W, int E, int N, int K, const int8_t* lut16, int lut_c, int ew,
                                             void* wq, void* sfw, void* wo, void* meta, void* stream, osc_weights** out) {
    return nvfp4_prepare_impl(W, E, N, K, K, lut16, lut_c, ew, wq, sfw, wo, meta, stream, out, true);
}

osc_status osc_nvfp4_act_sizes(const osc_weights* w, int M, osc_act_sizes_t* out) {
    if (!w || !out) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (!w->nvfp4) return fail(OSC_ERR_INVALID_ARG, "MXFP4 weights: use osc_act_sizes");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    const int64_t max_tiles = w->grouped ? (int64_t)M / 128 + w->E : ((int64_t)M + 127) / 128;
    out->xq_bytes = (size_t)M * (w->K / 2);
    out->sfa_bytes = (size_t)max_tiles * (w->K / 64) * 512;
    out->xo_bytes = (size_t)M * w->Kop * 2;
    out->sched_bytes = w->grouped ? sched_ints(max_tiles) * 4 + sched_ints(max_tiles256(M, w->E)) * 4 : 0;
    out->xq_offset = 0;
    out->sfa_offset = out->xq_offset + align256(out->xq_bytes);
    out->xo_offset = out->sfa_offset + align256(out->sfa_bytes);
    out->sched_offset = out->xo_offset + align256(out->xo_bytes);
    out->workspace_bytes = out->sched_offset + align256(out->sched_bytes);
    return OSC_OK;
}

static osc_status nvfp4_quantize_impl(const osc_weights* w, const void* X, int M, int64_t ldx, int ex, void* xq, void* sfa,
                                      void* xo, void* stream, const int32_t* sched, int max_tiles) {
    if (osc_status s = check_act(w, X, M, ldx, false, true)) return s;
    if (ex < -100 || ex > 100) return fail(OSC_ERR_INVALID_ARG, "tensor exponent %d outside -100..100", ex);
    if (M == 0) return OSC_OK;
    if (!xq || !sfa || (w->Kop > 0 && !xo)) return fail(OSC_ERR_INVALID_ARG, "null output pointer");
    if (!aligned16(xq) || !aligned16(sfa) || !aligned16(xo)) return fail(OSC_ERR_ALIGN, "outputs must be 16-byte aligned");
    CUtensorMap tm_x;
    if (osc_status s = make_tmap_x(&tm_x, X, M, w->K, ldx)) return s;
    cudaError_t e = launch_quant_extract_nvfp4(tm_x, M, w->K, w->mask, w->prefix, w->idx_o, xq, sfa, w->Kop ? xo : nullptr,
                                               w->Ko, w->Kop, w->num_sms, ex, static_cast<cudaStream_t>(stream), sched, max_tiles);
    if (e != cudaSuccess) return cuda_fail(e, "quant_extract_kernel(nvfp4)");
    return OSC_OK;
}
osc_status osc_nvfp4_quantize_extract(const osc_weights* w, const void* X, int M, int64_t ldx, int ex, void* xq,
                                      void* sfa, void* xo, void* stream) {
    if (w && w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_nvfp4_linear_grouped");
    return nvfp4_quantize_impl(w, X, M, ldx, ex, xq, sfa, xo, stream, nullptr, 0);
}

static osc_status nvfp4_gemm_impl(const osc_weights* w, const void* xq, const void* sfa, const void* xo, int M, int ex, void* Y,
                                  int64_t ldy, void* stream, const int32_t* sched, int max_tiles, const int32_t* sched2,
                                  int max_tiles2) {
    if (!w) return fail(OSC_ERR_INVALID_ARG, "weights handle is null");
    if (!w->nvfp4) return fail(OSC_ERR_INVALID_ARG, "MXFP4 weights: use osc_gemm_dual");
    if (M < 0) return fail(OSC_ERR_INVALID_ARG, "M = %d is negative", M);
    if (M == 0) return OSC_OK;
    if (!xq || !sfa || !Y || (w->Kop > 0 && !xo)) return fail(OSC_ERR_INVALID_ARG, "null device pointer");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y) || !aligned16(xq) || !aligned16(sfa) || !aligned16(xo))
        return fail(OSC_ERR_ALIGN, "pointers must be 16-byte aligned and ldy a multiple of 8");
    const int es = ex + w->ew;
    if (es < -120 || es > 120) return fail(OSC_ERR_INVALID_ARG, "sum of the tensor exponents %d outside -120..120", es);
    GemmArgs a;
    memset(&a, 0, sizeof a);
    const int nkb = (w->K + 255) / 256 + w->Kop / 64;
    if (use_decode_kernel(w->grouped, M, w->N, nkb, w->num_sms, true)) {   // few rows: weights stream once, K split over a cluster
        const uint32_t tok_box = (uint32_t)((M + 15) / 16 * 16);
        if (osc_status s = make_tmap(&a.tm_a, xq, false, M, w->K / 2, w->K / 2, tok_box)) return s;
        a.tm_b = w->tm_b[1];
        if (w->Kop > 0) {
            if (osc_status s = make_tmap(&a.tm_ao, xo, true, M, (uint64_t)w->Kop * 2, (uint64_t)w->Kop * 2, tok_box)) return s;
            a.tm_bo = w->tm_bo[1];
        }
        a.sfa = static_cast<const uint8_t*>(sfa);
        a.sfw = w->sfw;
        a.Y = static_cast<uint16_t*>(Y);
        a.ldy = ldy;
        a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
        a.num_sms = w->num_sms;
        a.out_scale = ldexpf(1.0f, es);
        cudaError_t e = launch_gemm_nvf4_decode(a, gemm_decode_split(w->N, nkb, w->num_sms), static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "gemm_decode_kernel(nvfp4)");
        return OSC_OK;
    }
    if (osc_status s = make_tmap(&a.tm_a, xq, false, M, w->K / 2, w->K / 2, 128)) return s;
    long single_ns = 0, pair_ns = 0;
    const int bn1 = gemm_block_n(sched ? max_tiles : (M + 127) / 128, w->N, w->num_sms, &single_ns, 192);
    const long row_tiles2 = w->grouped ? (max_tiles2 > w->E / 2 ? max_tiles2 - w->E / 2 : 1) : (M + 255) / 256;
    const int bn = gemm_pair_block_n(false, !w->grouped, row_tiles2, w->N, nkb, w->num_sms, &pair_ns);
    a.sched = sched; a.max_tiles = max_tiles;
    a.sched2 = sched2; a.max_tiles2 = max_tiles2;
    if (!use_pair_kernel(w->grouped, M, w->E, single_ns * nkb, pair_ns, single_ns <= 390)) {   // 128-row tiles
        a.tm_b = w->tm_b[bn1 / 64 - 1];
        if (w->Kop > 0) {
            if (osc_status s = make_tmap(&a.tm_ao, xo, true, M, (uint64_t)w->Kop * 2, (uint64_t)w->Kop * 2, 128)) return s;
            a.tm_bo = w->tm_bo[bn1 / 64 - 1];
        }
        a.sfa = static_cast<const uint8_t*>(sfa);
        a.sfw = w->sfw;
        a.Y = static_cast<uint16_t*>(Y);
        a.ldy = ldy;
        a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
        a.num_sms = w->num_sms;
        a.out_scale = ldexpf(1.0f, es);
        cudaError_t e = launch_gemm_nvf4(a, bn1, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "gemm_kernel(nvfp4)");
        return OSC_OK;
    }
    const int v2 = bn == 192 ? 0 : bn == 256 ? 1 : 2;
    a.tm_b = w->tm_b2[v2];
    if (w->Kop > 0) {
        if (osc_status s = make_tmap(&a.tm_ao, xo, true, M, (uint64_t)w->Kop * 2, (uint64_t)w->Kop * 2, 128)) return s;
        a.tm_bo = w->tm_bo2[v2];
    }
    a.tm_sfw = (bn == kTiledBN) ? w->tm_sfw_tiled : w->tm_sfw;
    const uint64_t sf_row_blocks = w->grouped ? (uint64_t)max_tiles : (uint64_t)((M + 127) / 128);
    if (osc_status s = make_tmap_sf(&a.tm_sfa, sfa, sf_row_blocks * (w->K / 64), 4)) return s;
    if (osc_status s = make_tmap(&a.tm_y, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 32)) return s;
    if (osc_status s = make_tmap(&a.tm_y16, Y, true, M, (uint64_t)w->N * 2, (uint64_t)ldy * 2, 16)) return s;
    a.sfa = static_cast<const uint8_t*>(sfa);
    a.sfw = w->sfw;
    a.Y = static_cast<uint16_t*>(Y);
    a.ldy = ldy;
    a.M = M; a.N = w->N; a.K = w->K; a.Kop = w->Kop;
    a.num_sms = w->num_sms;
    a.out_scale = ldexpf(1.0f, es);
    cudaError_t e = launch_gemm_nvf4_pair(a, bn, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "gemm_pair_kernel(nvfp4)");
    return OSC_OK;
}

osc_status osc_nvfp4_gemm(const osc_weights* w, const void* xq, const void* sfa, const void* xo, int M, int ex, void* Y,
                          int64_t ldy, void* stream) {
    if (w && w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_nvfp4_linear_grouped");
    return nvfp4_gemm_impl(w, xq, sfa, xo, M, ex, Y, ldy, stream, nullptr, 0, nullptr, 0);
}

osc_status osc_nvfp4_linear_grouped(const osc_weights* w, const void* X_perm, const int32_t* off, int M_total, int64_t ldx,
                                    int ex, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X_perm, M_total, ldx, false, true)) return s;
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights: use osc_nvfp4_linear");
    if (ex < -100 || ex > 100) return fail(OSC_ERR_INVALID_ARG, "tensor exponent %d outside -100..100", ex);
    if (M_total == 0) return OSC_OK;
    if (!off) return fail(OSC_ERR_INVALID_ARG, "off is null");
    osc_act_sizes_t sz;
    osc_nvfp4_act_sizes(w, M_total, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    const int es = ex + w->ew;
    if (es < -120 || es > 120) return fail(OSC_ERR_INVALID_ARG, "sum of the tensor exponents %d outside -120..120", es);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int max_tiles = M_total / 128 + w->E;
    const int max_tiles2 = max_tiles256(M_total, w->E);
    int32_t* sched = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
    int32_t* sched2 = use_pair_kernel(true, M_total, w->E) ? sched + sched_ints(max_tiles) : nullptr;
    cudaError_t e = launch_build_sched(off, w->E, sched, max_tiles, sched2, max_tiles2, st);
    if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
    if (osc_status s = nvfp4_quantize_impl(w, X_perm, M_total, ldx, ex, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset,
                                           stream, sched, max_tiles)) return s;
    return nvfp4_gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M_total, ex, Y, ldy, stream, sched,
                           max_tiles, sched2, max_tiles2);
}

// ---- NVFP4 forms of the producer fusion and of the dispatch gather
static osc_status nvfp4_rmsnorm_quantize_impl(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma,
                                              float eps, int ex, void* xq, void* sfa, void* xo, void* stream) {
    if (osc_status s = check_act(w, H, M, ldh, false, true)) return s;
    if (ex < -100 || ex > 100) return fail(OSC_ERR_INVALID_ARG, "tensor exponent %d outside -100..100", ex);
    if (w->K > 8192) return fail(OSC_ERR_SHAPE, "K = %d: the fused RMSNorm stages a row in shared memory, K <= 8192", w->K);
    if (M == 0) return OSC_OK;
    if (!gamma || !aligned16(gamma)) return fail(OSC_ERR_ALIGN, "gamma must be non-null and 16-byte aligned");
    if (!xq || !sfa || (w->Kop > 0 && !xo)) return fail(OSC_ERR_INVALID_ARG, "null output pointer");
    if (!aligned16(xq) || !aligned16(sfa) || !aligned16(xo)) return fail(OSC_ERR_ALIGN, "outputs must be 16-byte aligned");
    cudaError_t e = launch_rmsnorm_quant_nvfp4(H, ldh, M, w->K, gamma, eps, w->idx_o, xq, sfa, w->Kop ? xo : nullptr, w->Ko,
                                               w->Kop, ex, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "rmsnorm_quant_kernel(nvfp4)");
    return OSC_OK;
}

osc_status osc_nvfp4_rmsnorm_quantize_extract(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma,
                                              float eps, int ex, void* xq, void* sfa, void* xo, void* stream) {
    if (w && w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_nvfp4_rmsnorm_linear_grouped_gather");
    return nvfp4_rmsnorm_quantize_impl(w, H, M, ldh, gamma, eps, ex, xq, sfa, xo, stream);
}

osc_status osc_nvfp4_rmsnorm_linear(const osc_weights* w, const void* H, int M, int64_t ldh, const void* gamma, float eps,
                                    int ex, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, H, M, ldh, false, true)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_nvfp4_rmsnorm_linear_grouped_gather");
    if (M == 0) return OSC_OK;
    osc_act_sizes_t sz;
    osc_nvfp4_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (osc_status s = nvfp4_rmsnorm_quantize_impl(w, H, M, ldh, gamma, eps, ex, ws + sz.xq_offset, ws + sz.sfa_offset,
                                                   ws + sz.xo_offset, stream)) return s;
    return osc_nvfp4_gemm(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M, ex, Y, ldy, stream);
}

// buffers of the T unique tokens behind the grouped workspace (NVFP4: scale blocks of 64 channels)
static GatherLayout nvfp4_gather_layout(const osc_weights* w, int T, const osc_act_sizes_t& sz) {
    GatherLayout g;
    g.xq_u = sz.workspace_bytes;
    g.sf_u = g.xq_u + align256((size_t)T * (w->K / 2));
    g.xo_u = g.sf_u + align256((size_t)((T + 127) / 128) * (w->K / 64) * 512);
    g.total = g.xo_u + align256((size_t)T * w->Kop * 2);
    return g;
}

osc_status osc_nvfp4_gather_workspace_bytes(const osc_weights* w, int T, int M_total, size_t* bytes) {
    if (!w || !bytes) return fail(OSC_ERR_INVALID_ARG, "null argument");
    if (!w->nvfp4) return fail(OSC_ERR_INVALID_ARG, "MXFP4 weights: use osc_gather_workspace_bytes");
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights have no dispatch");
    if (T < 0 || M_total < 0) return fail(OSC_ERR_INVALID_ARG, "negative size");
    osc_act_sizes_t sz;
    if (osc_status s = osc_nvfp4_act_sizes(w, M_total, &sz)) return s;
    *bytes = nvfp4_gather_layout(w, T, sz).total;
    return OSC_OK;
}

static osc_status nvfp4_grouped_gather_impl(const osc_weights* w, const void* X, int T, int64_t ldx, const void* gamma, float eps,
                                            const int32_t* row_token, const int32_t* off, int M_total, int ex, void* Y,
                                            int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, T, ldx, false, true)) return s;
    if (!w->grouped) return fail(OSC_ERR_INVALID_ARG, "dense weights have no dispatch");
    if (M_total < 0) return fail(OSC_ERR_INVALID_ARG, "M_total = %d is negative", M_total);
    if (ex < -100 || ex > 100) return fail(OSC_ERR_INVALID_ARG, "tensor exponent %d outside -100..100", ex);
    if (M_total == 0) return OSC_OK;
    if (T == 0) return fail(OSC_ERR_INVALID_ARG, "rows to dispatch but no tokens");
    if (!off || !row_token) return fail(OSC_ERR_INVALID_ARG, "off / row_token is null");
    osc_act_sizes_t sz;
    osc_nvfp4_act_sizes(w, M_total, &sz);
    const GatherLayout g = nvfp4_gather_layout(w, T, sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < g.total)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, g.total);
    if (!Y) return fail(OSC_ERR_INVALID_ARG, "Y is null");
    if (ldy < w->N) return fail(OSC_ERR_SHAPE, "ldy = %lld < N = %d", (long long)ldy, w->N);
    if (ldy % 8 || !aligned16(Y)) return fail(OSC_ERR_ALIGN, "Y must be 16-byte aligned and ldy a multiple of 8");
    const int es = ex + w->ew;
    if (es < -120 || es > 120) return fail(OSC_ERR_INVALID_ARG, "sum of the tensor exponents %d outside -120..120", es);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int max_tiles = M_total / 128 + w->E;
    const int max_tiles2 = max_tiles256(M_total, w->E);
    int32_t* sched = reinterpret_cast<int32_t*>(ws + sz.sched_offset);
    int32_t* sched2 = use_pair_kernel(true, M_total, w->E) ? sched + sched_ints(max_tiles) : nullptr;
    cudaError_t e = launch_build_sched(off, w->E, sched, max_tiles, sched2, max_tiles2, st);
    if (e != cudaSuccess) return cuda_fail(e, "build_sched_kernel");
    // the NVFP4 form of Algorithm 2 once per token, as a dense problem of T rows
    if (gamma) {
        if (osc_status s = nvfp4_rmsnorm_quantize_impl(w, X, T, ldx, gamma, eps, ex, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, stream))
            return s;
    } else {
        if (osc_status s = nvfp4_quantize_impl(w, X, T, ldx, ex, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, stream, nullptr, 0)) return s;
    }
    e = launch_gather_quantized(row_token, T, w->K, w->Kop, ws + g.xq_u, ws + g.sf_u, ws + g.xo_u, ws + sz.xq_offset,
                                ws + sz.sfa_offset, ws + sz.xo_offset, sched, max_tiles, st, 64);
    if (e != cudaSuccess) return cuda_fail(e, "gather_quantized_kernel(nvfp4)");
    return nvfp4_gemm_impl(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M_total, ex, Y, ldy, stream, sched,
                           max_tiles, sched2, max_tiles2);
}

osc_status osc_nvfp4_linear_grouped_gather(const osc_weights* w, const void* X, int T, int64_t ldx, const int32_t* row_token,
                                           const int32_t* off, int M_total, int ex, void* Y, int64_t ldy, void* workspace,
                                           size_t workspace_bytes, void* stream) {
    return nvfp4_grouped_gather_impl(w, X, T, ldx, nullptr, 0.0f, row_token, off, M_total, ex, Y, ldy, workspace, workspace_bytes,
                                     stream);
}

osc_status osc_nvfp4_rmsnorm_linear_grouped_gather(const osc_weights* w, const void* H, int T, int64_t ldh, const void* gamma,
                                                   float eps, const int32_t* row_token, const int32_t* off, int M_total, int ex,
                                                   void* Y, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
    if (!gamma) return fail(OSC_ERR_INVALID_ARG, "gamma is null");
    return nvfp4_grouped_gather_impl(w, H, T, ldh, gamma, eps, row_token, off, M_total, ex, Y, ldy, workspace, workspace_bytes,
                                     stream);
}

osc_status osc_nvfp4_linear(const osc_weights* w, const void* X, int M, int64_t ldx, int ex, void* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* stream) {
    if (osc_status s = check_act(w, X, M, ldx, false, true)) return s;
    if (w->grouped) return fail(OSC_ERR_INVALID_ARG, "grouped weights: use osc_nvfp4_linear_grouped");
    if (M == 0) return OSC_OK;
    osc_act_sizes_t sz;
    osc_nvfp4_act_sizes(w, M, &sz);
    if (!workspace || !aligned16(workspace)) return fail(OSC_ERR_ALIGN, "workspace must be non-null and 16-byte aligned");
    if (workspace_bytes < sz.workspace_bytes)
        return fail(OSC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, sz.workspace_bytes);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (osc_status s = osc_nvfp4_quantize_extract(w, X, M, ldx, ex, ws + sz.xq_offset, ws + sz.sfa_offset,
                                                  ws + sz.xo_offset, stream)) return s;
    return osc_nvfp4_gemm(w, ws + sz.xq_offset, ws + sz.sfa_offset, ws + sz.xo_offset, M, ex, Y, ldy, stream);
}

}  // extern "C"
