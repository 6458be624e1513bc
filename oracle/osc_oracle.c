/*
 * CPU oracle for the OSC dual-path quantized linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * CUDA library must compute; only the test-suite, the smoke check and the
 * bench's cpu-baseline leg may call it.  It shares no code, table or header
 * with the CUDA path.
 *
 * What it follows:
 *   - Algorithm 2 (OSC-enhanced quantization): reshape to [S, K, G], look up the
 *     suppression indices, back the flagged channels up into the buffer B, zero
 *     them, CalculateScale, Quantize.
 *   - Eq. 5 (dual-path GEMM): Y = (Q_X (x) Q_W) . S  +  B . W_L.
 *   - Section 3.3 "offline weight quantization": W pre-quantized to FP4 and the
 *     high-precision weight rows W_L gathered with the same table.
 *   - Section 3.4 (hybrid-precision fallback): FP8 W8A8 linear for W2 inputs.
 *   - "Standard micro-scaling" (Algorithm 2, CalculateScale / Quantize) is read as
 *     the OCP Microscaling v1.0 MXFP4 definition the paper cites: group of 32,
 *     shared scale 2^(floor(log2(amax)) - 2) stored as E8M0, elements E2M1 with
 *     round-to-nearest-even and saturation.
 *
 * All floating point is done in double, on values that are exactly
 * representable (bf16 inputs, power-of-two scales), except where the FP8
 * per-token scale is *defined* in fp32 (see osc_ref_fp8_quantize).
 * bf16 tensors are passed as uint16 bit patterns.
 *
 * Pins (tests/test_oracle_*.py): E2M1/E4M3 tables against an independent
 * library codec, closed-form scale codes, the worked 32-element vectors under
 * tests/golden/, empty-table and full-table reductions against a numpy double
 * GEMM, brute force on tiny shapes, restoration identity, error ordering;
 * the MXFP8 fallback against a numpy + library-codec restatement, its own worked
 * group and a dense product of the dequantized operands.
 * Unpinned: nothing in this file (the paper's accuracy tables are out of scope).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define G 32 /* micro-scaling group size (MXFP4) */

/* ------------------------------------------------------------------ scalars */

static double bf16_value(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* The eight non-negative E2M1 magnitudes, code 0..7 (OCP MX v1.0, FP4 E2M1). */
static const double E2M1_MAG[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

double osc_ref_e2m1_decode(int nibble) {
    double m = E2M1_MAG[nibble & 7];
    return (nibble & 8) ? -m : m;
}

/* Nearest E2M1 value, ties to the even code, |v| > 6 saturates to 6; the sign bit
 * of v is kept even when the magnitude rounds to zero. NaN maps to +6. */
int osc_ref_e2m1_encode(double v) {
    if (isnan(v)) return 7;
    int sign = signbit(v) ? 8 : 0;
    double a = fabs(v);
    int best = 0;
    double bestd = INFINITY;
    for (int c = 0; c < 8; ++c) {
        double d = fabs(a - E2M1_MAG[c]);
        if (d < bestd || (d == bestd && (c % 2 == 0))) {
            bestd = d;
            best = c;
        }
    }
    if (a > 6.0) best = 7;
    return sign | best;
}

/* E8M0 code of the shared scale of one group: 2^(floor(log2 amax) - emax), with
 * emax(E2M1) = 2, clamped to the E8M0 range [2^-127, 2^127]; a group of zeros
 * takes the smallest scale; a non-finite amax gives the NaN code 0xFF. */
int osc_ref_e8m0_from_amax(double amax) {
    if (isnan(amax) || isinf(amax)) return 0xFF;
    if (amax == 0.0) return 0;
    int ex;
    (void)frexp(amax, &ex); /* amax = m * 2^ex, m in [0.5,1)  =>  floor(log2 amax) = ex-1 */
    int code = (ex - 1) - 2 + 127;
    if (code < 0) code = 0;
    if (code > 254) code = 254;
    return code;
}

/* E4M3 (OCP FP8, "FN": no infinity, max finite 448) value of a 7-bit magnitude code. */
static double e4m3_mag(int code) {
    int e = (code >> 3) & 15, m = code & 7;
    if (e == 0) return ldexp((double)m, -9);         /* subnormals: m * 2^-9 */
    return ldexp(1.0 + (double)m / 8.0, e - 7);
}

double osc_ref_e4m3_decode(int byte) {
    int c = byte & 0x7F;
    if (c == 0x7F) return NAN;
    double m = e4m3_mag(c);
    return (byte & 0x80) ? -m : m;
}

/* Nearest finite E4M3 value (codes 0x00..0x7E), ties to the even code, saturating
 * at 448; sign bit kept. NaN maps to 0x7F. */
int osc_ref_e4m3_encode(double v) {
    if (isnan(v)) return 0x7F;
    int sign = signbit(v) ? 0x80 : 0;
    double a = fabs(v);
    int best = 0;
    double bestd = INFINITY;
    for (int c = 0; c <= 0x7E; ++c) {
        double d = fabs(a - e4m3_mag(c));
        if (d < bestd || (d == bestd && (c % 2 == 0))) {
            bestd = d;
            best = c;
        }
    }
    if (a > 448.0) best = 0x7E;
    return sign | best;
}

/* ------------------------------------------------------ scale-factor layout */

/* Byte offset of the scale of (row r, group g) for a tensor with K columns:
 * 512-byte blocks of 128 rows x 4 groups, blocks ordered row-block major then
 * along K; inside a block byte = (r%32)*16 + ((r%128)/32)*4 + g%4. */
int64_t osc_ref_sf_index(int64_t r, int64_t g, int64_t K) {
    int64_t kblocks = K / 128;
    return ((r / 128) * kblocks + g / 4) * 512 + (r % 32) * 16 + ((r % 128) / 32) * 4 + (g % 4);
}

int64_t osc_ref_sf_bytes(int64_t rows, int64_t K) {
    return ((rows + 127) / 128) * (K / 128) * 512;
}

/* ---------------------------------------------------------- lookup table */

/* Normalise the suppression table of one layer/position: lut[Kg][C], entries in
 * -1..31 (-1 = no channel). Produces the per-group bit mask, the running count
 * of flagged channels before each group, and the ascending channel list.
 * Returns K_o >= 0, or -1 for an entry out of range, -2 for a duplicate. */
int osc_ref_lut_normalize(const int8_t* lut, int Kg, int C, uint32_t* mask, int32_t* prefix,
                          int32_t* idx_o) {
    int Ko = 0;
    for (int k = 0; k < Kg; ++k) {
        uint32_t m = 0;
        for (int c = 0; c < C; ++c) {
            int j = lut[(int64_t)k * C + c];
            if (j < -1 || j >= G) return -1;
            if (j < 0) continue;
            if (m & (1u << j)) return -2;
            m |= 1u << j;
        }
        mask[k] = m;
        prefix[k] = Ko;
        for (int j = 0; j < G; ++j)
            if (m & (1u << j)) idx_o[Ko++] = k * G + j;
    }
    return Ko;
}

int osc_ref_ko_pad(int Ko) { return (Ko + 63) / 64 * 64; }

/* --------------------------------------------- Algorithm 2 on one tensor */

/* Rows of X (bf16 bits, leading dimension ldx) -> packed E2M1 codes xq [M, K/2],
 * E8M0 scales in the block layout (sf, rows of this call start at SF row 0), and
 * the buffer B of backed-up channels xo [M, K_o_pad] (bf16 bits; pad columns +0).
 * The same routine serves the offline weight split (rows of W). */
int osc_ref_quantize_extract(const uint16_t* X, int64_t ldx, int M, int K, const int8_t* lut, int C,
                             uint8_t* xq, uint8_t* sf, uint16_t* xo) {
    if (K % G) return -3;
    int Kg = K / G;
    uint32_t* mask = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)Kg);
    int32_t* prefix = (int32_t*)malloc(sizeof(int32_t) * (size_t)Kg);
    int32_t* idx_o = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    int Ko = osc_ref_lut_normalize(lut, Kg, C, mask, prefix, idx_o);
    if (Ko < 0) { free(mask); free(prefix); free(idx_o); return Ko; }
    int Kop = osc_ref_ko_pad(Ko);

#pragma omp parallel for schedule(static)
    for (int s = 0; s < M; ++s) {
        const uint16_t* xrow = X + (int64_t)s * ldx;
        double xr[G];
        int nib[G];
        /* buffer B starts as zeros */
        for (int t = 0; t < Kop; ++t) xo[(int64_t)s * Kop + t] = 0;
        for (int k = 0; k < Kg; ++k) {
            /* X_reshaped[s, k, :] */
            for (int j = 0; j < G; ++j) xr[j] = bf16_value(xrow[k * G + j]);
            /* back up and zero the flagged channels of this group */
            int t = prefix[k];
            for (int j = 0; j < G; ++j) {
                if (mask[k] & (1u << j)) {
                    xo[(int64_t)s * Kop + t] = xrow[k * G + j];
                    ++t;
                    xr[j] = 0.0;
                }
            }
            /* CalculateScale */
            double amax = 0.0;
            for (int j = 0; j < G; ++j) {
                double a = fabs(xr[j]);
                if (a > amax || isnan(a)) amax = a;
            }
            int code = osc_ref_e8m0_from_amax(amax);
            sf[osc_ref_sf_index(s, k, K)] = (uint8_t)code;
            /* Quantize: element / scale, scale = 2^(code-127) (a division by a power of two is exact) */
            for (int j = 0; j < G; ++j) nib[j] = osc_ref_e2m1_encode(ldexp(xr[j], 127 - code));
            for (int i = 0; i < G / 2; ++i)
                xq[(int64_t)s * (K / 2) + k * (G / 2) + i] = (uint8_t)(nib[2 * i] | (nib[2 * i + 1] << 4));
        }
    }
    free(mask); free(prefix); free(idx_o);
    return Ko;
}

/* Grouped form: token rows sorted by expert, expert e owns rows [off[e], off[e+1]);
 * its scales start at SF row sum_{e'<e} roundup(m_e', 128). */
int64_t osc_ref_sf_row_base(const int32_t* off, int E, int64_t* base) {
    int64_t b = 0;
    for (int e = 0; e < E; ++e) {
        base[e] = b;
        b += ((int64_t)(off[e + 1] - off[e]) + 127) / 128 * 128;
    }
    return b;
}

int osc_ref_quantize_extract_grouped(const uint16_t* X, int64_t ldx, const int32_t* off, int E, int K,
                                     const int8_t* lut, int C, uint8_t* xq, uint8_t* sf, uint16_t* xo,
                                     int Kop) {
    int64_t* base = (int64_t*)malloc(sizeof(int64_t) * (size_t)(E > 0 ? E : 1));
    osc_ref_sf_row_base(off, E, base);
    int rc = 0;
    for (int e = 0; e < E; ++e) {
        int m = off[e + 1] - off[e];
        rc = osc_ref_quantize_extract(X + (int64_t)off[e] * ldx, ldx, m, K, lut, C,
                                      xq + (int64_t)off[e] * (K / 2),
                                      sf + (base[e] / 128) * (K / 128) * 512,
                                      xo + (int64_t)off[e] * Kop);
        if (rc < 0) break;
    }
    free(base);
    return rc;
}

/* --------------------------------------------------------- Eq. 5, dual path */

/* For the listed activation rows (rows[i] indexes xq/xo, sf_rows[i] indexes the
 * scale buffer) and all N weight rows:
 *   Y[i][n] = sum_g 2^(sa-127) 2^(sw-127) sum_{c in g} a[c] w[c]   (Path A)
 *           + sum_t xo[t] wo[t]                                     (Path B)
 *   T[i][n] = the same sums over absolute values (scale of the error bound).
 * Every product is exact in double; sums run in index order. */
int osc_ref_gemm_dual_rows(const uint8_t* xq, const uint8_t* sfa, const uint16_t* xo,
                           const int32_t* rows, const int32_t* sf_rows, int nrows,
                           const uint8_t* wq, const uint8_t* sfw, const uint16_t* wo,
                           int N, int K, int Kop, double* Y, double* T) {
    int Kg = K / G;
    /* decode the selected activation rows once */
    double* a = (double*)malloc(sizeof(double) * (size_t)nrows * (size_t)(K > 0 ? K : 1));
    int* sa = (int*)malloc(sizeof(int) * (size_t)nrows * (size_t)(Kg > 0 ? Kg : 1));
    double* b = (double*)malloc(sizeof(double) * (size_t)nrows * (size_t)(Kop > 0 ? Kop : 1));
    for (int i = 0; i < nrows; ++i) {
        int64_t r = rows[i];
        for (int c = 0; c < K; ++c) {
            int byte = xq[r * (K / 2) + c / 2];
            a[(int64_t)i * K + c] = osc_ref_e2m1_decode((c & 1) ? (byte >> 4) : (byte & 15));
        }
        for (int g = 0; g < Kg; ++g) sa[(int64_t)i * Kg + g] = sfa[osc_ref_sf_index(sf_rows[i], g, K)];
        for (int t = 0; t < Kop; ++t) b[(int64_t)i * Kop + t] = bf16_value(xo[r * Kop + t]);
    }
#pragma omp parallel
    {
        double* w = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
        double* wl = (double*)malloc(sizeof(double) * (size_t)(Kop > 0 ? Kop : 1));
        int* sw = (int*)malloc(sizeof(int) * (size_t)(Kg > 0 ? Kg : 1));
#pragma omp for schedule(static)
        for (int n = 0; n < N; ++n) {
            for (int c = 0; c < K; ++c) {
                int byte = wq[(int64_t)n * (K / 2) + c / 2];
                w[c] = osc_ref_e2m1_decode((c & 1) ? (byte >> 4) : (byte & 15));
            }
            for (int g = 0; g < Kg; ++g) sw[g] = sfw[osc_ref_sf_index(n, g, K)];
            for (int t = 0; t < Kop; ++t) wl[t] = bf16_value(wo[(int64_t)n * Kop + t]);
            for (int i = 0; i < nrows; ++i) {
                const double* ai = a + (int64_t)i * K;
                const int* sai = sa + (int64_t)i * Kg;
                double acc = 0.0, tot = 0.0;
                for (int g = 0; g < Kg; ++g) {
                    double p = 0.0, q = 0.0;
                    for (int c = g * G; c < (g + 1) * G; ++c) {
                        double pr = ai[c] * w[c];
                        p += pr;
                        q += fabs(pr);
                    }
                    int e = sai[g] + sw[g] - 254;
                    acc += ldexp(p, e);
                    tot += ldexp(q, e);
                }
                const double* bi = b + (int64_t)i * Kop;
                for (int t = 0; t < Kop; ++t) {
                    double pr = bi[t] * wl[t];
                    acc += pr;
                    tot += fabs(pr);
                }
                Y[(int64_t)i * N + n] = acc;
                T[(int64_t)i * N + n] = tot;
            }
        }
        free(w); free(wl); free(sw);
    }
    free(a); free(sa); free(b);
    return 0;
}

/* ------------------------------------------------- FP8 fallback (Section 3.4) */

/* Per-row dynamic E4M3: amax' = max(amax, 2^-40); sx = amax'/448 and
 * inv = 448/amax' (fp32 divisions), code = E4M3(fl32(x * inv)).  The scale
 * arithmetic is fixed to fp32 because it decides integer codes. */
int osc_ref_fp8_quantize(const uint16_t* X, int64_t ldx, int M, int K, uint8_t* x8, float* sx) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t* xrow = X + (int64_t)m * ldx;
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = fabsf((float)bf16_value(xrow[k]));
            if (a > amax) amax = a;
        }
        float floor_ = ldexpf(1.0f, -40);
        volatile float amaxp = amax > floor_ ? amax : floor_;
        volatile float s = amaxp / 448.0f;
        volatile float inv = 448.0f / amaxp;
        sx[m] = s;
        for (int k = 0; k < K; ++k) {
            volatile float v = (float)bf16_value(xrow[k]) * inv;
            x8[(int64_t)m * K + k] = (uint8_t)osc_ref_e4m3_encode((double)v);
        }
    }
    return 0;
}

/* Y[i][n] = sx[r] sw[n] sum_k q_x q_w ; T = same with absolute values. */
int osc_ref_fp8_gemm_rows(const uint8_t* x8, const float* sx, const int32_t* rows, int nrows,
                          const uint8_t* w8, const float* sw, int N, int K, double* Y, double* T) {
    double* a = (double*)malloc(sizeof(double) * (size_t)nrows * (size_t)(K > 0 ? K : 1));
    for (int i = 0; i < nrows; ++i)
        for (int k = 0; k < K; ++k) a[(int64_t)i * K + k] = osc_ref_e4m3_decode(x8[(int64_t)rows[i] * K + k]);
#pragma omp parallel
    {
        double* w = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(static)
        for (int n = 0; n < N; ++n) {
            for (int k = 0; k < K; ++k) w[k] = osc_ref_e4m3_decode(w8[(int64_t)n * K + k]);
            for (int i = 0; i < nrows; ++i) {
                const double* ai = a + (int64_t)i * K;
                double acc = 0.0, tot = 0.0;
                for (int k = 0; k < K; ++k) {
                    double pr = ai[k] * w[k];
                    acc += pr;
                    tot += fabs(pr);
                }
                double s = (double)sx[rows[i]] * (double)sw[n];
                Y[(int64_t)i * N + n] = s * acc;
                T[(int64_t)i * N + n] = s * tot;
            }
        }
        free(w);
    }
    free(a);
    return 0;
}

/* ----------------- NVFP4 / G = 16 variant (Section 3.3 efficiency table, G = 16 row; Section 5) */

/* The paper reports OSC on NVFP4 as well (blocks of 16, Table "Hardware Efficiency" row G = 16) without
 * giving the arithmetic; this is the reading used here.  NVFP4 = E2M1 elements in blocks of 16 along K, one
 * unsigned E4M3 scale per block, one tensor-level scale.  The tensor-level scale is restricted to a power of
 * two, 2^e, so that the high-precision branch can live in the same scaled domain exactly:
 *   x' = x * 2^-e                       (exact)
 *   per block b (after the flagged channels are backed up and zeroed, as in Algorithm 2 with G = 16):
 *     t  = fl32(amax_b' * fl32(1/6))                     amax_b' = max |x'| over the block
 *     sb = E4M3_rne_sat(t)                               stored scale byte (0x00..0x7E)
 *     q  = E2M1_rne_sat(fl32(x' * fl32(1 / value(sb))))  if value(sb) > 0, else the sign-only zero code
 *   backed-up channels: xo = x' rounded to bf16 (exact while x' is a normal bf16 number)
 * The scale arithmetic is fp32 because it decides integer codes.  Scale bytes use the 128 x 4 block layout
 * with one 512-byte block per 128 rows x 64 channels (four 16-blocks):
 *   byte(r, b) = ((r/128)*(K/64) + b/4)*512 + (r%32)*16 + ((r%128)/32)*4 + b%4,  b = block index along K. */
#define G16 16

int64_t osc_ref_sf16_index(int64_t r, int64_t b, int64_t K) {
    return ((r / 128) * (K / 64) + b / 4) * 512 + (r % 32) * 16 + ((r % 128) / 32) * 4 + (b % 4);
}
int64_t osc_ref_sf16_bytes(int64_t rows, int64_t K) { return ((rows + 127) / 128) * (K / 64) * 512; }

/* table for 16-groups: lut[K/16][C], entries -1..15.  Same outputs as osc_ref_lut_normalize with one 16-bit
 * mask per 16-group. Returns K_o, -1 (range) or -2 (duplicate). */
int osc_ref_lut16_normalize(const int8_t* lut, int Kg, int C, uint32_t* mask, int32_t* prefix, int32_t* idx_o) {
    int Ko = 0;
    for (int k = 0; k < Kg; ++k) {
        uint32_t m = 0;
        for (int c = 0; c < C; ++c) {
            int j = lut[(int64_t)k * C + c];
            if (j < -1 || j >= G16) return -1;
            if (j < 0) continue;
            if (m & (1u << j)) return -2;
            m |= 1u << j;
        }
        mask[k] = m;
        prefix[k] = Ko;
        for (int j = 0; j < G16; ++j)
            if (m & (1u << j)) idx_o[Ko++] = k * G16 + j;
    }
    return Ko;
}

/* bf16 bits of the value v * 2^-e rounded to bf16 (nearest even): exact whenever the result is a normal
 * bf16 number, i.e. always for the tensor scales a calibration would pick. */
static uint16_t bf16_scale_pow2(uint16_t b, int e) {
    float f = (float)ldexp(bf16_value(b), -e); /* exact: 8 significant bits, fp32 exponent range */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7F800000u) == 0x7F800000u) return (uint16_t)(u >> 16); /* non-finite: truncated */
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

int osc_ref_nvfp4_quantize_extract(const uint16_t* X, int64_t ldx, int M, int K, const int8_t* lut, int C, int e,
                                   uint8_t* xq, uint8_t* sf, uint16_t* xo) {
    if (K % 64) return -3;
    int Kg = K / G16;
    uint32_t* mask = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)Kg);
    int32_t* prefix = (int32_t*)malloc(sizeof(int32_t) * (size_t)Kg);
    int32_t* idx_o = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    int Ko = osc_ref_lut16_normalize(lut, Kg, C, mask, prefix, idx_o);
    if (Ko < 0) { free(mask); free(prefix); free(idx_o); return Ko; }
    int Kop = osc_ref_ko_pad(Ko);
    volatile float sixth = 1.0f / 6.0f;

#pragma omp parallel for schedule(static)
    for (int s = 0; s < M; ++s) {
        const uint16_t* xrow = X + (int64_t)s * ldx;
        for (int t = 0; t < Kop; ++t) xo[(int64_t)s * Kop + t] = 0;
        for (int k = 0; k < Kg; ++k) {
            float xr[G16];
            int nib[G16];
            for (int j = 0; j < G16; ++j) xr[j] = (float)ldexp(bf16_value(xrow[k * G16 + j]), -e); /* exact */
            int t = prefix[k];
            for (int j = 0; j < G16; ++j) {
                if (mask[k] & (1u << j)) {
                    xo[(int64_t)s * Kop + t] = bf16_scale_pow2(xrow[k * G16 + j], e);
                    ++t;
                    xr[j] = 0.0f;
                }
            }
            float amax = 0.0f;
            for (int j = 0; j < G16; ++j) {
                float a = fabsf(xr[j]);
                if (a > amax) amax = a;
            }
            volatile float tt = amax * sixth;
            int sb = osc_ref_e4m3_encode((double)tt) & 0x7F;
            sf[osc_ref_sf16_index(s, k, K)] = (uint8_t)sb;
            float sbv = (float)osc_ref_e4m3_decode(sb);
            volatile float inv = sbv > 0.0f ? 1.0f / sbv : 0.0f;
            for (int j = 0; j < G16; ++j) {
                volatile float v = xr[j] * inv;
                nib[j] = osc_ref_e2m1_encode((double)v);
            }
            for (int i = 0; i < G16 / 2; ++i)
                xq[(int64_t)s * (K / 2) + k * (G16 / 2) + i] = (uint8_t)(nib[2 * i] | (nib[2 * i + 1] << 4));
        }
    }
    free(mask); free(prefix); free(idx_o);
    return Ko;
}

/* Y[i][n] = 2^(ex+ew) * ( sum_b sa*sw * sum_{c in b} a[c] w[c]  +  sum_t xo[t] wo[t] ), T likewise with
 * absolute values; sa, sw = the E4M3 block scales. */
int osc_ref_nvfp4_gemm_rows(const uint8_t* xq, const uint8_t* sfa, const uint16_t* xo, const int32_t* rows, int nrows,
                            const uint8_t* wq, const uint8_t* sfw, const uint16_t* wo, int N, int K, int Kop,
                            int e_sum, double* Y, double* T) {
    int Kb = K / G16;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int i = 0; i < nrows; ++i) {
            int64_t r = rows[i];
            double acc = 0.0, tot = 0.0;
            for (int b = 0; b < Kb; ++b) {
                double p = 0.0, q = 0.0;
                for (int c = b * G16; c < (b + 1) * G16; ++c) {
                    int xa = xq[r * (K / 2) + c / 2], wa = wq[(int64_t)n * (K / 2) + c / 2];
                    double pr = osc_ref_e2m1_decode((c & 1) ? (xa >> 4) : (xa & 15)) *
                                osc_ref_e2m1_decode((c & 1) ? (wa >> 4) : (wa & 15));
                    p += pr;
                    q += fabs(pr);
                }
                double sc = osc_ref_e4m3_decode(sfa[osc_ref_sf16_index(r, b, K)]) *
                            osc_ref_e4m3_decode(sfw[osc_ref_sf16_index(n, b, K)]);
                acc += sc * p;
                tot += sc * q;
            }
            for (int t = 0; t < Kop; ++t) {
                double pr = bf16_value(xo[r * Kop + t]) * bf16_value(wo[(int64_t)n * Kop + t]);
                acc += pr;
                tot += fabs(pr);
            }
            Y[(int64_t)i * N + n] = ldexp(acc, e_sum);
            T[(int64_t)i * N + n] = ldexp(tot, e_sum);
        }
    }
    return 0;
}

/* ---------------- dynamic-protection baseline (Section 4.2, "OSC vs. Optimized Dynamic Protection") */

/* The control group the paper compares against: per token and per 32-group the
 * element of largest magnitude is found AT RUN TIME, kept in high precision and
 * removed before the group is scaled and quantized (same CalculateScale /
 * Quantize as Algorithm 2).  Ties take the lowest channel; an all-zero group
 * "extracts" its first element (a zero).  Outputs per row m and group g:
 * idx[m][g] = local channel 0..31, val[m][g] = the bf16 element (bit copy);
 * xq / sf as in osc_ref_quantize_extract.  The weights of this baseline are
 * quantized whole (no column is zeroed: any column can be picked by some token). */
int osc_ref_dyn_quantize_extract(const uint16_t* X, int64_t ldx, int M, int K, uint8_t* xq, uint8_t* sf,
                                 uint8_t* idx, uint16_t* val) {
    int Kg = K / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t* xrow = X + (int64_t)m * ldx;
        for (int g = 0; g < Kg; ++g) {
            int best = 0;
            double bestv = -1.0;
            for (int j = 0; j < G; ++j) {
                double a = fabs(bf16_value(xrow[g * G + j]));
                if (a > bestv) {
                    bestv = a;
                    best = j;
                }
            }
            idx[(int64_t)m * Kg + g] = (uint8_t)best;
            val[(int64_t)m * Kg + g] = xrow[g * G + best];
            double amax = 0.0;
            for (int j = 0; j < G; ++j) {
                if (j == best) continue;
                double a = fabs(bf16_value(xrow[g * G + j]));
                if (a > amax) amax = a;
            }
            int code = osc_ref_e8m0_from_amax(amax);
            sf[osc_ref_sf_index(m, g, K)] = (uint8_t)code;
            for (int j = 0; j < G; j += 2) {
                int nib[2];
                for (int t = 0; t < 2; ++t) {
                    uint16_t b = (j + t == best) ? (uint16_t)0 : xrow[g * G + j + t];
                    nib[t] = osc_ref_e2m1_encode(ldexp(bf16_value(b), 127 - code));
                }
                xq[(int64_t)m * (K / 2) + (g * G + j) / 2] = (uint8_t)(nib[0] | (nib[1] << 4));
            }
        }
    }
    return 0;
}

/* ------------------------- MXFP8 fallback (Section 3.4; Section 4 "Implementation Details") */

/* The 8-bit micro-scaling form of the W2 fallback: groups of 32 along K share an
 * E8M0 scale 2^(floor(log2 amax) - emax) with emax(E4M3) = 8 (OCP MX v1.0, MXFP8
 * E4M3), elements are E4M3 with round-to-nearest-even and saturation at 448.
 * No channel is extracted: the fallback applies to inputs whose outliers are
 * diffuse.  Scales go to the same 128 x 4 block layout as the MXFP4 scales. */
int osc_ref_e8m0_from_amax_emax(double amax, int emax) {
    if (isnan(amax) || isinf(amax)) return 0xFF;
    if (amax == 0.0) return 0;
    int ex;
    (void)frexp(amax, &ex); /* floor(log2 amax) = ex - 1 */
    int code = (ex - 1) - emax + 127;
    if (code < 0) code = 0;
    if (code > 254) code = 254;
    return code;
}

int osc_ref_mxfp8_quantize(const uint16_t* X, int64_t ldx, int M, int K, uint8_t* x8, uint8_t* sf) {
    int Kg = K / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t* xrow = X + (int64_t)m * ldx;
        for (int g = 0; g < Kg; ++g) {
            double amax = 0.0;
            for (int c = g * G; c < (g + 1) * G; ++c) {
                double a = fabs(bf16_value(xrow[c]));
                if (a > amax || isnan(a)) amax = a;
            }
            int code = osc_ref_e8m0_from_amax_emax(amax, 8);
            sf[osc_ref_sf_index(m, g, K)] = (uint8_t)code;
            for (int c = g * G; c < (g + 1) * G; ++c) {
                double v = ldexp(bf16_value(xrow[c]), 127 - code); /* exact: power-of-two scaling */
                x8[(int64_t)m * K + c] = (uint8_t)osc_ref_e4m3_encode(v);
            }
        }
    }
    return 0;
}

/* Y[i][n] = sum_g 2^(sa-127) 2^(sw-127) sum_{c in g} a[c] w[c] over E4M3 elements;
 * T = the same with absolute values.  Products are exact in double. */
int osc_ref_mxfp8_gemm_rows(const uint8_t* x8, const uint8_t* sfa, const int32_t* rows, int nrows,
                            const uint8_t* w8, const uint8_t* sfw, int N, int K, double* Y, double* T) {
    int Kg = K / G;
    double* a = (double*)malloc(sizeof(double) * (size_t)nrows * (size_t)(K > 0 ? K : 1));
    int* sa = (int*)malloc(sizeof(int) * (size_t)nrows * (size_t)(Kg > 0 ? Kg : 1));
    for (int i = 0; i < nrows; ++i) {
        int64_t r = rows[i];
        for (int c = 0; c < K; ++c) a[(int64_t)i * K + c] = osc_ref_e4m3_decode(x8[r * K + c]);
        for (int g = 0; g < Kg; ++g) sa[(int64_t)i * Kg + g] = sfa[osc_ref_sf_index(r, g, K)];
    }
#pragma omp parallel
    {
        double* w = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
        int* sw = (int*)malloc(sizeof(int) * (size_t)(Kg > 0 ? Kg : 1));
#pragma omp for schedule(static)
        for (int n = 0; n < N; ++n) {
            for (int c = 0; c < K; ++c) w[c] = osc_ref_e4m3_decode(w8[(int64_t)n * K + c]);
            for (int g = 0; g < Kg; ++g) sw[g] = sfw[osc_ref_sf_index(n, g, K)];
            for (int i = 0; i < nrows; ++i) {
                const double* ai = a + (int64_t)i * K;
                const int* sai = sa + (int64_t)i * Kg;
                double acc = 0.0, tot = 0.0;
                for (int g = 0; g < Kg; ++g) {
                    double p = 0.0, q = 0.0;
                    for (int c = g * G; c < (g + 1) * G; ++c) {
                        double pr = ai[c] * w[c];
                        p += pr;
                        q += fabs(pr);
                    }
                    int e = sai[g] + sw[g] - 254;
                    acc += ldexp(p, e);
                    tot += ldexp(q, e);
                }
                Y[(int64_t)i * N + n] = acc;
                T[(int64_t)i * N + n] = tot;
            }
        }
        free(w); free(sw);
    }
    free(a); free(sa);
    return 0;
}

/* ------------------------------------------- offline profiling (Section 2, Algorithm 1) */

/* ---- SwiGLU in front of the per-token FP8 quantizer (the producer of the down projection's input; Section 3.3
 * places the quantizer directly behind the operator that produces the activations, Section 3.4 makes that
 * quantizer FP8 for this input).  The paper does not give the activation's arithmetic; it is fixed here in
 * fp32, every step an IEEE operation, so that the FP8 codes that follow are decided on identical values:
 *
 *   exp32(z):  t = fl32(z * LOG2E) clamped to [-64, 126] (beyond, 1 + e is 1 or the quotient g / (1 + e) is
 *              below 1e-35 in magnitude: nothing a bf16 product with u can show);
 *              n = rint(t) (ties to even), f = t - n (exact), p = Horner with fused multiply-adds of the
 *              degree-5 Taylor polynomial of 2^f on [-1/2, 1/2]; e = p * 2^n (exact scaling)
 *   silu32(g) = fl32( g * fl32( 1 / fl32(1 + exp32(-g)) ) )
 *   h = bf16( fl32( silu32(g) * u ) )        g = GU[m][i], u = GU[m][I + i]
 */
static const float OSC_EXP2_C[6] = {1.0f, 0.693147182f, 0.240226507f, 0.0555041097f, 0.00961812865f, 0.00133335579f};
float osc_ref_exp32(float z) {
    volatile float t = z * 1.44269502f;
    t = fminf(fmaxf(t, -64.0f), 126.0f); /* a NaN argument ends at -64: the NaN reaches the result through g itself */
    float n = rintf(t);
    float f = t - n;
    float p = OSC_EXP2_C[5];
    for (int i = 4; i >= 0; --i) p = fmaf(p, f, OSC_EXP2_C[i]);
    return ldexpf(p, (int)n);
}
float osc_ref_silu32(float g) {
    volatile float d = 1.0f + osc_ref_exp32(-g);
    volatile float r = 1.0f / d;
    volatile float s = g * r;
    return s;
}
static uint16_t bf16_from_float_rne(float v) {
    uint32_t u;
    memcpy(&u, &v, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FFF; /* NaN */
    return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}
int osc_ref_swiglu(const uint16_t* GU, int64_t ldg, int M, int I, uint16_t* H) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t* row = GU + (int64_t)m * ldg;
        for (int i = 0; i < I; ++i) {
            float g = (float)bf16_value(row[i]), u = (float)bf16_value(row[I + i]);
            volatile float hv = osc_ref_silu32(g) * u;
            H[(int64_t)m * I + i] = bf16_from_float_rne(hv);
        }
    }
    return 0;
}


/* Eq. 1: layer-wise threshold T_l = alpha * mean |x| over the S x H calibration activations. */
double osc_ref_threshold(const uint16_t* X, int64_t ldx, int S, int H, double alpha) {
    double sum = 0.0;
    for (int s = 0; s < S; ++s)
        for (int j = 0; j < H; ++j) sum += fabs(bf16_value(X[(int64_t)s * ldx + j]));
    return alpha * (sum / ((double)S * (double)H));
}

/* Largest bf16 magnitude (bit pattern, sign clear) whose value is <= T: for bf16 inputs |x| > T is the
 * same as bits(|x|) > this pattern, which makes the outlier test an integer comparison. */
uint32_t osc_ref_threshold_bits(double T) {
    if (!(T > 0.0)) return 0;
    float f = (float)T;
    if ((double)f > T) f = nextafterf(f, 0.0f);
    uint32_t u;
    memcpy(&u, &f, 4);
    return u >> 16;
}

/* Algorithm 1 for one (position, layer).  Per group the tokens vote: a token's vote is the local index of its
 * largest magnitude (the first one among equals), and it only counts when that magnitude exceeds the
 * layer's threshold.  The table entry of the group is the index with the most votes (the smallest such
 * index; -1 when nobody voted).  The vote counts also give Eq. 3-4: n_total = votes cast in the group,
 * n_hit = votes for the winning index, clustering density C = n_hit / n_total. */
static int strongest_channel(const uint16_t* group, double* magnitude) {
    int arg = 0;
    double top = fabs(bf16_value(group[0]));
    for (int j = 1; j < G; ++j) {
        const double a = fabs(bf16_value(group[j]));
        if (a > top) { top = a; arg = j; }
    }
    *magnitude = top;
    return arg;
}

int osc_ref_profile_indexing(const uint16_t* X, int64_t ldx, int S, int H, double T, int8_t* L, int32_t* n_hit,
                             int32_t* n_total) {
    if (H % G) return -3;
    const int groups = H / G;
    int32_t* votes = (int32_t*)calloc((size_t)groups * G, sizeof(int32_t));   /* votes[group][local index] */
    if (!votes) return -4;
    for (int s = 0; s < S; ++s) {
        const uint16_t* token = X + (int64_t)s * ldx;
        for (int k = 0; k < groups; ++k) {
            double magnitude;
            const int j = strongest_channel(token + k * G, &magnitude);
            if (magnitude > T) votes[k * G + j] += 1;
        }
    }
    for (int k = 0; k < groups; ++k) {
        const int32_t* v = votes + k * G;
        int winner = -1;
        int32_t cast = 0, won = 0;
        for (int j = 0; j < G; ++j) {
            cast += v[j];
            if (v[j] > won) { won = v[j]; winner = j; }
        }
        L[k] = (int8_t)winner;
        n_hit[k] = won;
        n_total[k] = cast;
    }
    free(votes);
    return 0;
}

int osc_ref_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
