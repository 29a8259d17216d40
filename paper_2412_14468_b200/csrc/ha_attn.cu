// GATHER-ATT (Section 4) and dense single-query SDPA (Section 3.1) as a split-K flash-decode pair:
// the partial kernel walks a slice of the index list (or of the whole sequence), reading the
// 256-byte bf16 K and V rows in place (Section 4.4: no gather into a separate buffer), and keeps an
// online-softmax state (running max, sum, unnormalised output) per query head in fp32; the
// combine kernel merges the slices' states and rounds once to bf16.
//
// All G query heads of a KV head are served by the same CTA so that every K/V row is read once.
#include "ha_common.cuh"

#include <math_constants.h>

namespace ha {

constexpr int kAttnWarps = 4;
constexpr int kAttnThreads = kAttnWarps * 32;
constexpr int kTokBatch = 4;   // rows in flight per warp
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void unpack4(uint2 r, float (&f)[4]) {
    f[0] = __uint_as_float(r.x << 16);
    f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16);
    f[3] = __uint_as_float(r.y & 0xffff0000u);
}

// One CTA = one slice of `split_tokens` list entries of one (sequence, KV head).
// Lane l owns dimensions 4l..4l+3 of every row; each warp walks its share of the slice.
template <int G, bool kGather>
__global__ void __launch_bounds__(kAttnThreads) attn_partial_kernel(
    const uint16_t *__restrict__ q, TensorView K, TensorView V, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, long long idx_sb, long long idx_sh, const int32_t *__restrict__ count,
    int max_items, int Hq, int Hkv, float scale_log2, int split_tokens, float *__restrict__ part_ml,
    float *__restrict__ part_acc, uint32_t *__restrict__ status) {
    __shared__ float s_m[kAttnWarps][G], s_l[kAttnWarps][G];
    __shared__ float s_acc[kAttnWarps][G][kD];

    const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int n = seq_lens[b];
    const int cnt = min(kGather ? count[b * Hkv + g] : n, max_items);
    const int start = split * split_tokens;
    if (start >= cnt) return;
    const int end = min(cnt, start + split_tokens);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    float qf[G][4];
#pragma unroll
    for (int j = 0; j < G; ++j) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(q + ((long long)b * Hq + g * G + j) * kD) + lane);
        unpack4(raw, qf[j]);
    }
    float m[G], l[G], acc[G][4];
#pragma unroll
    for (int j = 0; j < G; ++j) {
        m[j] = -CUDART_INF_F;
        l[j] = 0.0f;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][e] = 0.0f;
    }

    const uint16_t *Kb = K.ptr + (long long)b * K.sb + (long long)g * K.sh;
    const uint16_t *Vb = V.ptr + (long long)b * V.sb + (long long)g * V.sh;
    const int32_t *list = kGather ? idx + (long long)b * idx_sb + (long long)g * idx_sh : nullptr;

    for (int t0 = start + warp * kTokBatch; t0 < end; t0 += kAttnWarps * kTokBatch) {
        int tok[kTokBatch];
        uint2 kr[kTokBatch], vr[kTokBatch];
#pragma unroll
        for (int u = 0; u < kTokBatch; ++u) {
            int t = -1;
            if (t0 + u < end) {
                t = kGather ? __ldg(list + t0 + u) : (t0 + u);
                if (t >= n) {
                    if (lane == 0) atomicOr(status, HA_DEV_BAD_INDEX);
                    t = -1;
                }
            }
            tok[u] = t;
            if (t >= 0) {
                kr[u] = __ldg(reinterpret_cast<const uint2 *>(Kb + (long long)t * K.sn) + lane);
                vr[u] = __ldg(reinterpret_cast<const uint2 *>(Vb + (long long)t * V.sn) + lane);
            } else {
                kr[u] = make_uint2(0, 0);
                vr[u] = make_uint2(0, 0);
            }
        }
#pragma unroll
        for (int u = 0; u < kTokBatch; ++u) {
            if (tok[u] < 0) continue;   // uniform across the warp
            float kf[4], vf[4];
            unpack4(kr[u], kf);
            unpack4(vr[u], vf);
            float s[G];
#pragma unroll
            for (int j = 0; j < G; ++j) {
                float d = qf[j][0] * kf[0];
                d = fmaf(qf[j][1], kf[1], d);
                d = fmaf(qf[j][2], kf[2], d);
                d = fmaf(qf[j][3], kf[3], d);
                s[j] = d;
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1)
#pragma unroll
                for (int j = 0; j < G; ++j) s[j] += __shfl_xor_sync(0xffffffffu, s[j], off);
#pragma unroll
            for (int j = 0; j < G; ++j) {
                const float sj = s[j] * scale_log2;
                const float mn = fmaxf(m[j], sj);
                const float corr = exp2f(m[j] - mn);   // m = -inf on the first token: exp2(-inf) = 0
                const float p = exp2f(sj - mn);
                l[j] = fmaf(l[j], corr, p);
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[j][e] = fmaf(acc[j][e], corr, p * vf[e]);
                m[j] = mn;
            }
        }
    }

    // merge the warps of this CTA
#pragma unroll
    for (int j = 0; j < G; ++j) {
        if (lane == 0) { s_m[warp][j] = m[j]; s_l[warp][j] = l[j]; }
#pragma unroll
        for (int e = 0; e < 4; ++e) s_acc[warp][j][lane * 4 + e] = acc[j][e];
    }
    __syncthreads();
    const int d = threadIdx.x;   // kAttnThreads == kD
#pragma unroll
    for (int j = 0; j < G; ++j) {
        float M = s_m[0][j];
#pragma unroll
        for (int w = 1; w < kAttnWarps; ++w) M = fmaxf(M, s_m[w][j]);
        float L = 0.0f, A = 0.0f;
        if (M > -CUDART_INF_F) {
#pragma unroll
            for (int w = 0; w < kAttnWarps; ++w) {
                const float f = exp2f(s_m[w][j] - M);
                L = fmaf(s_l[w][j], f, L);
                A = fmaf(s_acc[w][j][d], f, A);
            }
        }
        const long long p = ((long long)b * Hq + g * G + j) * kMaxSplits + split;
        part_acc[p * kD + d] = A;
        if (d == 0) { part_ml[p * 2] = M; part_ml[p * 2 + 1] = L; }
    }
}

// Merge the slices of one query head: out = sum_s A_s 2^(M_s - M) / sum_s L_s 2^(M_s - M).
template <bool kGather>
__global__ void __launch_bounds__(kD) attn_combine_kernel(const int32_t *__restrict__ seq_lens,
                                                         const int32_t *__restrict__ count, int max_items, int Hq,
                                                         int Hkv, int split_tokens,
                                                         const float *__restrict__ part_ml,
                                                         const float *__restrict__ part_acc,
                                                         uint16_t *__restrict__ out, float *__restrict__ lse) {
    const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    const int g = h / (Hq / Hkv);
    const int cnt = min(kGather ? count[b * Hkv + g] : seq_lens[b], max_items);
    const int n_splits = (max(cnt, 0) + split_tokens - 1) / split_tokens;
    const long long p0 = ((long long)b * Hq + h) * kMaxSplits;
    float M = -CUDART_INF_F;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, part_ml[(p0 + s) * 2]);
    float L = 0.0f, A = 0.0f;
    if (M > -CUDART_INF_F) {
        for (int s = 0; s < n_splits; ++s) {
            const float f = exp2f(part_ml[(p0 + s) * 2] - M);
            L = fmaf(part_ml[(p0 + s) * 2 + 1], f, L);
            A = fmaf(part_acc[(p0 + s) * kD + d], f, A);
        }
    }
    const float o = (L > 0.0f) ? A / L : 0.0f;
    const __nv_bfloat16 ob = __float2bfloat16_rn(o);
    out[((long long)b * Hq + h) * kD + d] = *reinterpret_cast<const uint16_t *>(&ob);
    if (lse && d == 0) lse[b * Hq + h] = (L > 0.0f) ? (M * kLn2 + logf(L)) : -CUDART_INF_F;
}

int split_tokens_for(int n_units, int max_items) {
    // aim for about 8 CTAs per SM across the grid, at least 16 list entries per CTA,
    // at most kMaxSplits slices per unit
    const int target_ctas = 148 * 8;
    int splits = (target_ctas + n_units - 1) / max(n_units, 1);
    splits = max(1, min(splits, kMaxSplits));
    int tokens = (max(max_items, 1) + splits - 1) / splits;
    tokens = max(16, (tokens + 15) / 16 * 16);
    while ((max_items + tokens - 1) / tokens > kMaxSplits) tokens += 16;
    return tokens;
}

template <int G>
static cudaError_t launch_attn_g(bool gather, int B, int Hq, int Hkv, float sm_scale, const uint16_t *q,
                                 TensorView K, TensorView V, const int32_t *seq_lens, const int32_t *idx,
                                 long long idx_sb, long long idx_sh, const int32_t *count, int max_items,
                                 uint16_t *out, float *lse, float *part_ml, float *part_acc, uint32_t *status,
                                 cudaStream_t st) {
    const int split_tokens = split_tokens_for(B * Hkv, max_items);
    const int n_splits = max(1, (max_items + split_tokens - 1) / split_tokens);
    dim3 grid(n_splits, Hkv, B);
    const float scale_log2 = sm_scale * kLog2e;
    if (gather) {
        attn_partial_kernel<G, true><<<grid, kAttnThreads, 0, st>>>(q, K, V, seq_lens, idx, idx_sb, idx_sh, count,
                                                                    max_items, Hq, Hkv, scale_log2, split_tokens,
                                                                    part_ml, part_acc, status);
        attn_combine_kernel<true><<<dim3(Hq, B), kD, 0, st>>>(seq_lens, count, max_items, Hq, Hkv, split_tokens,
                                                              part_ml, part_acc, out, lse);
    } else {
        attn_partial_kernel<G, false><<<grid, kAttnThreads, 0, st>>>(q, K, V, seq_lens, idx, idx_sb, idx_sh, count,
                                                                     max_items, Hq, Hkv, scale_log2, split_tokens,
                                                                     part_ml, part_acc, status);
        attn_combine_kernel<false><<<dim3(Hq, B), kD, 0, st>>>(seq_lens, count, max_items, Hq, Hkv, split_tokens,
                                                               part_ml, part_acc, out, lse);
    }
    count_launch(2);
    return cudaGetLastError();
}

cudaError_t launch_attention(bool gather, int B, int Hq, int Hkv, float sm_scale, const uint16_t *q,
                             TensorView K, TensorView V, const int32_t *seq_lens, const int32_t *idx,
                             long long idx_sb, long long idx_sh, const int32_t *count, int max_items,
                             uint16_t *out, float *lse, float *part_ml, float *part_acc, uint32_t *status,
                             cudaStream_t st) {
#define HA_ARGS gather, B, Hq, Hkv, sm_scale, q, K, V, seq_lens, idx, idx_sb, idx_sh, count, max_items, out, lse, \
                part_ml, part_acc, status, st
    switch (Hq / Hkv) {
        case 1: return launch_attn_g<1>(HA_ARGS);
        case 2: return launch_attn_g<2>(HA_ARGS);
        case 4: return launch_attn_g<4>(HA_ARGS);
        case 8: return launch_attn_g<8>(HA_ARGS);
        default: return cudaErrorInvalidValue;
    }
#undef HA_ARGS
}

// Writes this step's new K and V rows into the cache at slot seq_len-1 (host-driven entry only).
__global__ void append_kv_kernel(int Hkv, const uint16_t *__restrict__ k_new, const uint16_t *__restrict__ v_new,
                                 TensorView K, TensorView V, const int32_t *__restrict__ seq_lens) {
    const int g = blockIdx.x, b = blockIdx.y, t = threadIdx.x;   // 32 threads x 8 bytes
    const int slot = seq_lens[b] - 1;
    if (slot < 0) return;
    const long long src = ((long long)b * Hkv + g) * kD;
    uint16_t *kd = const_cast<uint16_t *>(K.ptr) + (long long)b * K.sb + (long long)g * K.sh + (long long)slot * K.sn;
    uint16_t *vd = const_cast<uint16_t *>(V.ptr) + (long long)b * V.sb + (long long)g * V.sh + (long long)slot * V.sn;
    reinterpret_cast<uint2 *>(kd)[t] = reinterpret_cast<const uint2 *>(k_new + src)[t];
    reinterpret_cast<uint2 *>(vd)[t] = reinterpret_cast<const uint2 *>(v_new + src)[t];
}

cudaError_t launch_append_kv(int B, int Hkv, const uint16_t *k_new, const uint16_t *v_new, TensorView K,
                             TensorView V, const int32_t *seq_lens, cudaStream_t st) {
    append_kv_kernel<<<dim3(Hkv, B), 32, 0, st>>>(Hkv, k_new, v_new, K, V, seq_lens);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha
