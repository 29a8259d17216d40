// SCORE for wide signatures, and its inner-product comparator: the setting of the paper's table "Latency
// of SCORE computation" (one query against n cached tokens; signatures of 64 .. 512 bits kept as packed
// 64-bit integers, against the inner product with keys of 128 16-bit floats).  Eq. 1 with the bitcount
// identity of Section 4.1, at b bits: score = b - popc(k xor q).
//
// Both kernels are pure streams (8 .. 64 and 256 bytes per token in, 2 and 4 bytes out), bound by HBM:
// persistent CTAs, every lane reads 16 bytes per load with four loads in flight, a warp instruction covers
// 512 contiguous bytes.  A token of 256 or 512 bits is spread over 2 or 4 neighbouring lanes, whose partial
// counts meet through shuffles, so the loads stay contiguous whatever the width.
#include "ha_common.cuh"

namespace ha {

constexpr int kWideThreads = 256;
constexpr int kWideLoads = 4;   // 16-byte loads in flight per thread

// W = 64-bit words per signature (1, 2, 4, 8).  n16 = number of whole 16-byte pieces of the key array.
template <int W>
__global__ void __launch_bounds__(kWideThreads, (W == 2 || W == 4) ? 8 : 1) score_wide_kernel(const uint64_t *__restrict__ q_code,
                                                                 const uint64_t *__restrict__ k_codes, long long n,
                                                                 uint16_t *__restrict__ scores) {
    constexpr int kLanesPerToken = (W >= 2) ? W / 2 : 1;   // 16-byte pieces per token
    const int lane = threadIdx.x & 31;
    // the two query words that face this lane's 16-byte piece
    const int piece = lane % kLanesPerToken;
    const uint64_t qa = __ldg(q_code + ((W >= 2) ? 2 * piece : 0)), qb = __ldg(q_code + ((W >= 2) ? 2 * piece + 1 : 0));
    const long long n16 = (W >= 2) ? n * kLanesPerToken : n / 2;
    const uint4 *src = reinterpret_cast<const uint4 *>(k_codes);
    const long long per_iter = (long long)kWideThreads * kWideLoads;
    for (long long base = (long long)blockIdx.x * per_iter; base < n16; base += (long long)gridDim.x * per_iter) {
        uint4 v[kWideLoads];
#pragma unroll
        for (int j = 0; j < kWideLoads; ++j) {
            const long long i = base + (long long)j * kWideThreads + threadIdx.x;
            v[j] = (i < n16) ? __ldcs(src + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kWideLoads; ++j) {
            const long long i = base + (long long)j * kWideThreads + threadIdx.x;
            const unsigned long long lo = ((unsigned long long)v[j].y << 32) | v[j].x, hi = ((unsigned long long)v[j].w << 32) | v[j].z;
            const int da = __popcll(lo ^ qa), db = __popcll(hi ^ qb);
            if (W == 1) {   // two tokens in this piece
                if (i < n16) reinterpret_cast<uint32_t *>(scores)[i] = (uint32_t)(64 - da) | ((uint32_t)(64 - db) << 16);
            } else {
                int d = da + db;
                if (kLanesPerToken >= 2) d += __shfl_xor_sync(0xffffffffu, d, 1);
                if (kLanesPerToken >= 4) d += __shfl_xor_sync(0xffffffffu, d, 2);
                if (piece == 0 && i < n16) scores[i / kLanesPerToken] = (uint16_t)(64 * W - d);
            }
        }
    }
    if (W == 1 && (n & 1) && blockIdx.x == 0 && threadIdx.x == 0)   // odd count: the last token has no partner
        scores[n - 1] = (uint16_t)(64 - __popcll(__ldg(k_codes + n - 1) ^ qa));
}

// dots[i] = <q, K_i>, 128 bf16 components, fp32 accumulation: 16 lanes per row (eight components each).
__global__ void __launch_bounds__(kWideThreads, 8) inner_product_kernel(const uint16_t *__restrict__ q,
                                                                    const uint16_t *__restrict__ K, long long n,
                                                                    long long row_stride, float *__restrict__ dots) {
    const int lane = threadIdx.x & 31, part = lane & 15;
    float qf[8];
    {
        const uint4 qv = __ldg(reinterpret_cast<const uint4 *>(q) + part);
        const uint32_t w[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) { qf[2 * e] = __uint_as_float(w[e] << 16); qf[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
    }
    const long long rows_per_iter = (long long)kWideThreads / 16 * kWideLoads;   // 64 rows per CTA iteration
    for (long long base = (long long)blockIdx.x * rows_per_iter; base < n; base += (long long)gridDim.x * rows_per_iter) {
        uint4 v[kWideLoads];
#pragma unroll
        for (int j = 0; j < kWideLoads; ++j) {
            const long long r = base + (long long)j * (kWideThreads / 16) + (threadIdx.x >> 4);
            v[j] = (r < n) ? __ldcs(reinterpret_cast<const uint4 *>(K + r * row_stride) + part) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kWideLoads; ++j) {
            const long long r = base + (long long)j * (kWideThreads / 16) + (threadIdx.x >> 4);
            const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
            float acc = 0.0f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc = fmaf(__uint_as_float(w[e] << 16), qf[2 * e], acc);
                acc = fmaf(__uint_as_float(w[e] & 0xffff0000u), qf[2 * e + 1], acc);
            }
#pragma unroll
            for (int dd = 1; dd < 16; dd <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, dd);
            if (part == 0 && r < n) dots[r] = acc;
        }
    }
}

static int wide_grid(long long work_items, long long per_cta) {
    const long long want = (work_items + per_cta - 1) / per_cta;
    const long long cap = 8LL * sm_count();   // eight CTAs of 256 threads per SM
    return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

cudaError_t launch_score_wide(const uint64_t *q_code, const uint64_t *k_codes, long long n, int n_words, uint16_t *scores,
                              cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const long long pieces = (n_words >= 2) ? n * (n_words / 2) : (n + 1) / 2;
    const int grid = wide_grid(pieces, (long long)kWideThreads * kWideLoads);
    switch (n_words) {
        case 1: score_wide_kernel<1><<<grid, kWideThreads, 0, st>>>(q_code, k_codes, n, scores); break;
        case 2: score_wide_kernel<2><<<grid, kWideThreads, 0, st>>>(q_code, k_codes, n, scores); break;
        case 4: score_wide_kernel<4><<<grid, kWideThreads, 0, st>>>(q_code, k_codes, n, scores); break;
        case 8: score_wide_kernel<8><<<grid, kWideThreads, 0, st>>>(q_code, k_codes, n, scores); break;
        default: return cudaErrorInvalidValue;
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_inner_products(const uint16_t *q, const uint16_t *K, long long n, long long row_stride, float *dots,
                                  cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const int grid = wide_grid(n, (long long)kWideThreads / 16 * kWideLoads);
    inner_product_kernel<<<grid, kWideThreads, 0, st>>>(q, K, n, row_stride, dots);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha
