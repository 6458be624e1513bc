// Offline profiling of one (position, layer) activation slice: the layer-wise outlier threshold
// (Eq. 1), the per-token per-group argmax statistics (Eq. 2-4) and the suppression-table entries
// (Algorithm 1).  Not on the inference hot path; small, memory-bound kernels.
#include "common.cuh"

namespace osc {

// sum of |x| over the S x K slice, accumulated in fp64 (threads -> warp -> block -> one atomic per block)
__global__ void __launch_bounds__(256) profile_abs_sum_kernel(const uint16_t* __restrict__ X, int64_t ldx, int S,
                                                              int K, double* __restrict__ sum) {
    __shared__ double s_part[8];
    const int chunks_per_row = K / 8;
    const int64_t total = (int64_t)S * chunks_per_row;
    double acc = 0.0;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    constexpr int U = 4;   // independent 16-byte loads in flight per thread
    // (row, chunk) of the thread's next element, advanced without divisions
    const int64_t first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t r = first / chunks_per_row;
    int c = (int)(first - r * chunks_per_row);
    const int64_t dr = stride / chunks_per_row;
    const int dc = (int)(stride - dr * chunks_per_row);
    for (int64_t i0 = first; i0 < total; i0 += U * stride) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            v[u] = (i0 + u * stride < total) ? *reinterpret_cast<const uint4*>(X + r * ldx + c * 8) : make_uint4(0u, 0u, 0u, 0u);
            r += dr;
            c += dc;
            if (c >= chunks_per_row) { c -= chunks_per_row; ++r; }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {  // every magnitude enters the fp64 sum on its own (bf16 -> fp64 is exact)
                acc += (double)__uint_as_float((w[k] & 0x7FFFu) << 16);
                acc += (double)__uint_as_float(w[k] & 0x7FFF0000u);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < 8; ++i) t += s_part[i];
        atomicAdd(sum, t);
    }
}

// Largest bf16 magnitude pattern whose value is <= T (T > 0): |x| > T  <=>  bits(|x|) > pattern.
__device__ __forceinline__ uint32_t threshold_pattern(double T) {
    if (!(T > 0.0)) return 0u;
    return __float_as_uint(__double2float_rz(T)) >> 16;
}

// One thread per (token, group): first-maximum argmax over the 32 magnitudes; tokens whose maximum exceeds the
// threshold vote for their argmax channel.  A block owns PC_GROUPS consecutive groups and a slice of the tokens
// and collects its votes in shared memory (a channel that is an outlier in every token would otherwise take one
// global atomic per token on one address), then adds its 32 x PC_GROUPS counters to the global ones.
constexpr int PC_GROUPS = 8;
constexpr int PC_TOKENS = 128;   // tokens per block

__global__ void __launch_bounds__(256) profile_count_kernel(const uint16_t* __restrict__ X, int64_t ldx, int S, int K,
                                                            const double* __restrict__ sum, double alpha,
                                                            int32_t* __restrict__ counts,
                                                            uint32_t* __restrict__ threshold_bits) {
    __shared__ int s_counts[PC_GROUPS * 32];
    const int Kg = K / 32;
    const double T = alpha * (*sum / ((double)S * (double)K));
    const uint32_t tb = threshold_pattern(T);
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *threshold_bits = tb;
    for (int i = threadIdx.x; i < PC_GROUPS * 32; i += blockDim.x) s_counts[i] = 0;
    __syncthreads();
    const int gl = threadIdx.x % PC_GROUPS;            // my group inside the block's range
    const int k = blockIdx.x * PC_GROUPS + gl;
    const int s_end = min(S, ((int)blockIdx.y + 1) * PC_TOKENS);
    if (k < Kg) {
        for (int s0 = blockIdx.y * PC_TOKENS + threadIdx.x / PC_GROUPS; s0 < s_end; s0 += 256 / PC_GROUPS) {
            const uint16_t* p = X + (int64_t)s0 * ldx + k * 32;
            uint32_t best = 0;
            int jstar = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 v = *reinterpret_cast<const uint4*>(p + c * 8);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t lo = w[q] & 0x7FFFu, hi = (w[q] >> 16) & 0x7FFFu;
                    if (lo > best) { best = lo; jstar = c * 8 + 2 * q; }
                    if (hi > best) { best = hi; jstar = c * 8 + 2 * q + 1; }
                }
            }
            if (best > tb) atomicAdd(&s_counts[gl * 32 + jstar], 1);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < PC_GROUPS * 32; i += blockDim.x) {
        const int kk = blockIdx.x * PC_GROUPS + i / 32;
        if (kk < Kg && s_counts[i]) atomicAdd(&counts[kk * 32 + (i & 31)], s_counts[i]);
    }
}

// One thread per group: size of the candidate set, its most frequent index (smallest index among equals), -1 if empty.
__global__ void profile_finalize_kernel(const int32_t* __restrict__ counts, int Kg, int8_t* __restrict__ lut,
                                        int32_t* __restrict__ n_hit, int32_t* __restrict__ n_total) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= Kg) return;
    int total = 0, hit = 0, mode = -1;
    for (int j = 0; j < 32; ++j) {
        const int c = counts[k * 32 + j];
        total += c;
        if (c > hit) { hit = c; mode = j; }
    }
    lut[k] = (int8_t)(total > 0 ? mode : -1);
    n_hit[k] = hit;
    n_total[k] = total;
}

cudaError_t launch_profile(const void* X, int64_t ldx, int S, int K, double alpha, double* sum, int32_t* counts,
                           int8_t* lut, int32_t* n_hit, int32_t* n_total, uint32_t* threshold_bits, int num_sms,
                           cudaStream_t st) {
    const int Kg = K / 32;
    cudaError_t e = cudaMemsetAsync(sum, 0, 256 + (size_t)Kg * 32 * sizeof(int32_t), st);  // sum + counts are contiguous
    if (e != cudaSuccess) return e;
    const int64_t chunks = (int64_t)S * (K / 8);
    int g1 = (int)((chunks + 255) / 256 < 8L * num_sms ? (chunks + 255) / 256 : 8L * num_sms);
    if (g1 < 1) g1 = 1;
    profile_abs_sum_kernel<<<g1, 256, 0, st>>>(static_cast<const uint16_t*>(X), ldx, S, K, sum);
    const dim3 g2((Kg + PC_GROUPS - 1) / PC_GROUPS, (S + PC_TOKENS - 1) / PC_TOKENS);
    profile_count_kernel<<<g2, 256, 0, st>>>(static_cast<const uint16_t*>(X), ldx, S, K, sum, alpha, counts,
                                             threshold_bits);
    profile_finalize_kernel<<<(Kg + 127) / 128, 128, 0, st>>>(counts, Kg, lut, n_hit, n_total);
    return cudaGetLastError();
}

}  // namespace osc
