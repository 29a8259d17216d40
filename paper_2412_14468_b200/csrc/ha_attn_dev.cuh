// Device-side building blocks of the attention kernels (included by ha_attn.cu and ha_fused.cu).
#pragma once

#include "ha_common.cuh"

#include <math_constants.h>

namespace ha {

constexpr int kBlockTokens = 16;              // list entries per warp iteration
constexpr int kRowBytes = kD * 2 + 16;        // 256-byte row + 16 bytes so that ldmatrix rows hit distinct banks
constexpr int kTileBytes = kBlockTokens * kRowBytes;   // one block of K (or V) rows
constexpr int kStageBytes = 2 * kTileBytes;            // K tile followed by V tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte asynchronous global->shared copy; src_bytes = 0 writes zeros without reading
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
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


// Start the copies of one block (16 list entries) into a ring stage: half-warp h copies row 2r+h,
// lane%16 picks the 16-byte chunk, so each row is one 256-byte burst.  my_t = token id of list
// position lane%16 (-1: masked; its rows are zero-filled).  Returns the 16-bit validity mask.
__device__ __forceinline__ uint32_t attn_issue_block(uint32_t stage_u32, const unsigned char *Kb,
                                                     const unsigned char *Vb, long long k_row, long long v_row,
                                                     int my_t, int lane) {
    const uint32_t valid = __ballot_sync(0xffffffffu, my_t >= 0) & 0xffffu;
    const uint32_t kdst = stage_u32 + (lane >> 4) * kRowBytes + (lane & 15) * 16;
    const uint32_t vdst = kdst + kTileBytes;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const int t = __shfl_sync(0xffffffffu, my_t, 2 * r + (lane >> 4));
        const uint32_t nb = (t >= 0) ? 16u : 0u;
        const long long tt = (t >= 0) ? t : 0;
        cp_async16(kdst + r * 2 * kRowBytes, Kb + tt * k_row + (lane & 15) * 16, nb);
        cp_async16(vdst + r * 2 * kRowBytes, Vb + tt * v_row + (lane & 15) * 16, nb);
    }
    return valid;
}

// Query A fragments of head g = lane/4 (rows = heads, k = d); heads >= G are zero rows.
template <int G, bool kShared = false>
__device__ __forceinline__ void attn_load_q(uint32_t (&qa)[8][2], const uint16_t *q_group, int lane) {
    const int g = lane >> 2, c = lane & 3;
#pragma unroll
    for (int s = 0; s < 8; ++s) { qa[s][0] = 0u; qa[s][1] = 0u; }
    if (g < G) {
        const uint32_t *qp = reinterpret_cast<const uint32_t *>(q_group + (long long)g * kD);
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            if (kShared) { qa[s][0] = qp[8 * s + c]; qa[s][1] = qp[8 * s + c + 4]; }   // a copy in shared memory
            else { qa[s][0] = __ldg(qp + 8 * s + c); qa[s][1] = __ldg(qp + 8 * s + c + 4); }
        }
    }
}

// One block of 16 rows from a ring stage (K tile at ks, V tile at vs): S = Q K^T, online softmax for
// head g = lane/4, O^T += V^T P^T.  acc columns of this lane are heads 2c, 2c+1 (c = lane%4).
__device__ __forceinline__ void attn_consume_block(uint32_t ks, uint32_t vs, uint32_t valid,
                                                   const uint32_t (&qa)[8][2], float scale_log2, int lane,
                                                   float (&acc)[8][4], float &m_run, float &l_run) {
    const int c = lane & 3;
    // ldmatrix lane address: matrix j = lane/8 -> tokens (j/2)*8 + lane%8, 16-byte column block j%2
    const uint32_t lm_off = (((lane >> 4) << 3) + (lane & 7)) * kRowBytes + ((lane >> 3) & 1) * 16;

    // ---- S[head g][tokens 2c, 2c+1, 8+2c, 8+2c+1] = Q K^T
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        uint32_t kb[4];
        ldmatrix_x4(kb, ks + lm_off + s * 32);
        mma_bf16_16816(s0, qa[s][0], 0u, qa[s][1], 0u, kb[0], kb[1]);
        mma_bf16_16816(s1, qa[s][0], 0u, qa[s][1], 0u, kb[2], kb[3]);
    }

    // ---- online softmax for head g (log2 domain); masked entries contribute nothing
    float sv[4];
    sv[0] = ((valid >> (2 * c)) & 1u) ? s0[0] * scale_log2 : -CUDART_INF_F;
    sv[1] = ((valid >> (2 * c + 1)) & 1u) ? s0[1] * scale_log2 : -CUDART_INF_F;
    sv[2] = ((valid >> (2 * c + 8)) & 1u) ? s1[0] * scale_log2 : -CUDART_INF_F;
    sv[3] = ((valid >> (2 * c + 9)) & 1u) ? s1[1] * scale_log2 : -CUDART_INF_F;
    float bm = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
    const float m_new = fmaxf(m_run, bm);
    const float m_use = (m_new == -CUDART_INF_F) ? 0.0f : m_new;
    const float corr = exp2f(m_run - m_use);
    float p[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) p[e] = exp2f(sv[e] - m_use);
    l_run = fmaf(l_run, corr, (p[0] + p[1]) + (p[2] + p[3]));
    m_run = m_new;
    float ph[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) ph[e] = bf16_round(p[e]);
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

    // ---- O^T[d][head] += V^T P^T; the transposed ldmatrix pairs two tokens per register
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
        uint32_t va[4];
        ldmatrix_x4_trans(va, vs + lm_off + mt * 32);
        mma_bf16_16816(acc[mt], va[0], va[1], va[2], va[3], bh0, bh1);
        mma_bf16_16816(acc[mt], va[0], va[1], va[2], va[3], bl0, bl1);
    }
}

} // namespace ha
