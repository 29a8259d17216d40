// GATHER-ATT (Section 4) and dense single-query SDPA (Section 3.1) as one split-K flash-decode
// kernel.  A CTA owns a slice of the index list (or of the sequence) of one (sequence, KV head) and
// serves all G query heads of that KV head, so every selected K/V row is read from HBM once; the
// 256-byte bf16 rows are read in place through the indices (Section 4.4: no gather into a buffer).
//
// Data path per warp and per block of 16 list entries (8 KB of K/V rows, all loads issued before
// the first use so that a warp keeps 8 KB in flight):
//   * K rows go straight from global memory into mma.sync B fragments: four lanes share a row and
//     each takes 16-byte chunks, which fixes a permutation of the head dimension; the query
//     fragments are loaded with the same permutation, so the dot products are unchanged.
//   * S[head][token] = Q K^T on the tensor cores (m16n8k16, bf16 in, fp32 out), online softmax in
//     fp32 in the log2 domain; the C fragment of S is already the B fragment of P^T.
//   * V rows go from global memory into A fragments of V^T (two tokens are paired per register
//     with a byte permute), O^T[d][head] += V^T P^T with P split into bf16 hi + lo parts so that
//     the weights keep ~16 bits.
// The slices' states (running max, sum, unnormalised output) are merged by whichever CTA of the
// (sequence, KV head) finishes last (a ticket counter in the workspace; nobody waits), which
// normalises and rounds once to bf16.  The arithmetic intensity is ~4 FLOP/B: the kernel is bound
// by HBM, the tensor cores only keep the instruction count out of the way.
#include "ha_common.cuh"

#include <math_constants.h>

namespace ha {

constexpr int kAttnWarps = 4;
constexpr int kAttnThreads = kAttnWarps * 32;
constexpr int kBlockTokens = 16;   // list entries per warp iteration
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
    return *reinterpret_cast<const uint32_t *>(&v);
}

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

__device__ __forceinline__ uint32_t reg_of(const uint4 &v, int w) {
    return w == 0 ? v.x : (w == 1 ? v.y : (w == 2 ? v.z : v.w));
}

template <int G, bool kGather>
__global__ void __launch_bounds__(kAttnThreads, 3) attn_splitk_kernel(
    const uint16_t *__restrict__ q, TensorView K, TensorView V, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, long long idx_sb, long long idx_sh, const int32_t *__restrict__ count,
    int max_items, int Hq, int Hkv, float scale_log2, int split_tokens, float *__restrict__ part_ml,
    float *__restrict__ part_acc, int32_t *__restrict__ tickets, uint32_t *__restrict__ status,
    uint16_t *__restrict__ out, float *__restrict__ lse) {
    __shared__ float s_m[kAttnWarps][8], s_l[kAttnWarps][8];
    __shared__ float s_acc[kAttnWarps][G][kD];
    __shared__ int s_last;

    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int n = seq_lens[b];
    const int cnt = max(0, min(kGather ? count[b * Hkv + kvh] : n, max_items));
    const int n_splits = (cnt + split_tokens - 1) / split_tokens;
    const long long head0 = (long long)b * Hq + (long long)kvh * G;
    if (cnt == 0) {   // empty selection: out = 0, lse = -inf
        if (split == 0) {
            for (int i = tid; i < G * kD; i += kAttnThreads) out[head0 * kD + i] = 0;
            if (lse && tid < G) lse[head0 + tid] = -CUDART_INF_F;
        }
        return;
    }
    const int start = split * split_tokens;
    if (start >= cnt) return;
    const int end = min(cnt, start + split_tokens);

    // query fragments: lane (g, c) holds chunks 4i + c (16 bytes each) of head g's row, zero for g >= G
    uint4 qa[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) qa[i] = make_uint4(0, 0, 0, 0);
    if (g < G) {
        const uint4 *qp = reinterpret_cast<const uint4 *>(q + (head0 + g) * kD);
#pragma unroll
        for (int i = 0; i < 4; ++i) qa[i] = __ldg(qp + 4 * i + c);
    }

    float acc[8][4];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
    float m_run = -CUDART_INF_F, l_run = 0.0f;

    const uint16_t *Kb = K.ptr + (long long)b * K.sb + (long long)kvh * K.sh;
    const uint16_t *Vb = V.ptr + (long long)b * V.sb + (long long)kvh * V.sh;
    const int32_t *list = kGather ? idx + (long long)b * idx_sb + (long long)kvh * idx_sh : nullptr;
    bool bad = false;

    auto token_at = [&](int p) -> int {
        if (p >= end) return -1;
        int t = kGather ? __ldg(list + p) : p;
        if (t >= n) { bad = true; t = -1; }
        return t;
    };

    for (int p0 = start + warp * kBlockTokens; p0 < end; p0 += kAttnWarps * kBlockTokens) {
        // ---- which rows this lane fetches
        const int tk0 = token_at(p0 + g), tk1 = token_at(p0 + 8 + g);
        int tv[4];
        tv[0] = token_at(p0 + 2 * c);
        tv[1] = token_at(p0 + 2 * c + 1);
        tv[2] = token_at(p0 + 2 * c + 8);
        tv[3] = token_at(p0 + 2 * c + 9);

        // ---- issue every load of the block: K rows tk0, tk1 (chunks 4i+c), V rows tv[u] (chunks 8j+g)
        uint4 k0[4], k1[4], v[4][2];
        {
            const uint4 *kp0 = reinterpret_cast<const uint4 *>(Kb + (long long)max(tk0, 0) * K.sn);
            const uint4 *kp1 = reinterpret_cast<const uint4 *>(Kb + (long long)max(tk1, 0) * K.sn);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                k0[i] = (tk0 >= 0) ? ld_stream16(kp0 + 4 * i + c) : make_uint4(0, 0, 0, 0);
                k1[i] = (tk1 >= 0) ? ld_stream16(kp1 + 4 * i + c) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint4 *vp = reinterpret_cast<const uint4 *>(Vb + (long long)max(tv[u], 0) * V.sn);
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    v[u][j] = (tv[u] >= 0) ? ld_stream16(vp + 8 * j + g) : make_uint4(0, 0, 0, 0);
            }
        }

        // ---- S[head g][tokens 2c, 2c+1, 8+2c, 8+2c+1] = Q K^T
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_bf16_16816(s0, qa[i].x, 0u, qa[i].y, 0u, k0[i].x, k0[i].y);
            mma_bf16_16816(s0, qa[i].z, 0u, qa[i].w, 0u, k0[i].z, k0[i].w);
            mma_bf16_16816(s1, qa[i].x, 0u, qa[i].y, 0u, k1[i].x, k1[i].y);
            mma_bf16_16816(s1, qa[i].z, 0u, qa[i].w, 0u, k1[i].z, k1[i].w);
        }

        // ---- online softmax for head g (log2 domain); masked entries contribute nothing
        float sv[4];
        sv[0] = (tv[0] >= 0) ? s0[0] * scale_log2 : -CUDART_INF_F;
        sv[1] = (tv[1] >= 0) ? s0[1] * scale_log2 : -CUDART_INF_F;
        sv[2] = (tv[2] >= 0) ? s1[0] * scale_log2 : -CUDART_INF_F;
        sv[3] = (tv[3] >= 0) ? s1[1] * scale_log2 : -CUDART_INF_F;
        float bm = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
        const float m_new = fmaxf(m_run, bm);
        const float m_use = (m_new == -CUDART_INF_F) ? 0.0f : m_new;
        const float corr = exp2f(m_run - m_use);
        float p[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) p[u] = exp2f(sv[u] - m_use);
        l_run = fmaf(l_run, corr, (p[0] + p[1]) + (p[2] + p[3]));
        m_run = m_new;
        float ph[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) ph[u] = bf16_round(p[u]);
        const uint32_t bh0 = pack_bf16(ph[0], ph[1]), bh1 = pack_bf16(ph[2], ph[3]);
        const uint32_t bl0 = pack_bf16(p[0] - ph[0], p[1] - ph[1]), bl1 = pack_bf16(p[2] - ph[2], p[3] - ph[3]);

        // ---- rescale the running output when a maximum moved (columns of this lane: heads 2c, 2c+1)
        if (__any_sync(0xffffffffu, corr != 1.0f)) {
            const float ce = __shfl_sync(0xffffffffu, corr, (2 * c) * 4);
            const float co = __shfl_sync(0xffffffffu, corr, (2 * c + 1) * 4);
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                acc[mt][0] *= ce; acc[mt][1] *= co; acc[mt][2] *= ce; acc[mt][3] *= co;
            }
        }

        // ---- O^T[d][head] += V^T P^T : row-tile mt covers d = 8*rho + mt, rho = lane group (+8)
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            const int w = mt >> 1;
            const uint32_t sel = (mt & 1) ? 0x7632u : 0x5410u;
            const uint32_t a0 = __byte_perm(reg_of(v[0][0], w), reg_of(v[1][0], w), sel);
            const uint32_t a1 = __byte_perm(reg_of(v[0][1], w), reg_of(v[1][1], w), sel);
            const uint32_t a2 = __byte_perm(reg_of(v[2][0], w), reg_of(v[3][0], w), sel);
            const uint32_t a3 = __byte_perm(reg_of(v[2][1], w), reg_of(v[3][1], w), sel);
            mma_bf16_16816(acc[mt], a0, a1, a2, a3, bh0, bh1);
            mma_bf16_16816(acc[mt], a0, a1, a2, a3, bl0, bl1);
        }
    }
    if (bad) atomicOr(status, HA_DEV_BAD_INDEX);

    // ---- merge the warps of this CTA through shared memory
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (c == 0) { s_m[warp][g] = m_run; s_l[warp][g] = l_run; }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int h = 2 * c + hh;
        if (h < G) {
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                s_acc[warp][h][8 * g + mt] = acc[mt][hh];
                s_acc[warp][h][64 + 8 * g + mt] = acc[mt][2 + hh];
            }
        }
    }
    __syncthreads();
    const int d = tid;   // kAttnThreads == kD
    float Mj[G], Lj[G], Aj[G];
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
        Mj[j] = M; Lj[j] = L; Aj[j] = A;
    }

    if (n_splits > 1) {
        // publish this slice, take a ticket; the CTA that draws the last ticket merges all slices
#pragma unroll
        for (int j = 0; j < G; ++j) {
            const long long pidx = (head0 + j) * kMaxSplits + split;
            part_acc[pidx * kD + d] = Aj[j];
            if (d == 0) { part_ml[pidx * 2] = Mj[j]; part_ml[pidx * 2 + 1] = Lj[j]; }
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int t = atomicAdd(&tickets[b * Hkv + kvh], 1);
            s_last = (t == n_splits - 1);
            if (s_last) tickets[b * Hkv + kvh] = 0;   // ready for the next call
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
#pragma unroll
        for (int j = 0; j < G; ++j) {
            const long long p0 = (head0 + j) * kMaxSplits;
            float M = -CUDART_INF_F;
            for (int s = 0; s < n_splits; ++s) M = fmaxf(M, __ldcg(part_ml + (p0 + s) * 2));
            float L = 0.0f, A = 0.0f;
            if (M > -CUDART_INF_F) {
                for (int s = 0; s < n_splits; ++s) {
                    const float f = exp2f(__ldcg(part_ml + (p0 + s) * 2) - M);
                    L = fmaf(__ldcg(part_ml + (p0 + s) * 2 + 1), f, L);
                    A = fmaf(__ldcg(part_acc + (p0 + s) * kD + d), f, A);
                }
            }
            Mj[j] = M; Lj[j] = L; Aj[j] = A;
        }
    }
#pragma unroll
    for (int j = 0; j < G; ++j) {
        const float o = (Lj[j] > 0.0f) ? Aj[j] / Lj[j] : 0.0f;
        const __nv_bfloat16 ob = __float2bfloat16_rn(o);
        out[(head0 + j) * kD + d] = *reinterpret_cast<const uint16_t *>(&ob);
        if (lse && d == 0) lse[head0 + j] = (Lj[j] > 0.0f) ? (Mj[j] * kLn2 + logf(Lj[j])) : -CUDART_INF_F;
    }
}

int split_tokens_for(int n_units, int max_items) {
    // About four waves of 3 CTAs per SM when there is that much work, never fewer than 64 list
    // entries per CTA (one 16-entry block per warp), never more than kMaxSplits slices per unit.
    const long long total = (long long)max(n_units, 1) * max(max_items, 1);
    const long long target_ctas = 148LL * 3 * 4;
    long long tokens = (total + target_ctas - 1) / target_ctas;
    tokens = (tokens + kBlockTokens - 1) / kBlockTokens * kBlockTokens;
    if (tokens < kAttnWarps * kBlockTokens) tokens = kAttnWarps * kBlockTokens;
    while (((long long)max_items + tokens - 1) / tokens > kMaxSplits) tokens += kBlockTokens;
    return (int)tokens;
}

template <int G>
static cudaError_t launch_attn_g(bool gather, int B, int Hq, int Hkv, float sm_scale, const uint16_t *q,
                                 TensorView K, TensorView V, const int32_t *seq_lens, const int32_t *idx,
                                 long long idx_sb, long long idx_sh, const int32_t *count, int max_items,
                                 uint16_t *out, float *lse, float *part_ml, float *part_acc, int32_t *tickets,
                                 uint32_t *status, cudaStream_t st) {
    const int split_tokens = split_tokens_for(B * Hkv, max_items);
    const int n_splits = max(1, (max_items + split_tokens - 1) / split_tokens);
    dim3 grid(n_splits, Hkv, B);
    const float scale_log2 = sm_scale * kLog2e;
    if (gather)
        attn_splitk_kernel<G, true><<<grid, kAttnThreads, 0, st>>>(q, K, V, seq_lens, idx, idx_sb, idx_sh, count,
                                                                   max_items, Hq, Hkv, scale_log2, split_tokens,
                                                                   part_ml, part_acc, tickets, status, out, lse);
    else
        attn_splitk_kernel<G, false><<<grid, kAttnThreads, 0, st>>>(q, K, V, seq_lens, idx, idx_sb, idx_sh, count,
                                                                    max_items, Hq, Hkv, scale_log2, split_tokens,
                                                                    part_ml, part_acc, tickets, status, out, lse);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_attention(bool gather, int B, int Hq, int Hkv, float sm_scale, const uint16_t *q,
                             TensorView K, TensorView V, const int32_t *seq_lens, const int32_t *idx,
                             long long idx_sb, long long idx_sh, const int32_t *count, int max_items,
                             uint16_t *out, float *lse, float *part_ml, float *part_acc, int32_t *tickets,
                             uint32_t *status, cudaStream_t st) {
#define HA_ARGS gather, B, Hq, Hkv, sm_scale, q, K, V, seq_lens, idx, idx_sb, idx_sh, count, max_items, out, lse, \
                part_ml, part_acc, tickets, status, st
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
