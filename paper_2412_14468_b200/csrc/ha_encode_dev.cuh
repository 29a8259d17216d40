// Device-side building blocks of the decode-step ENCODE (included by ha_encode.cu and ha_fused.cu).
#pragma once

#include "ha_common.cuh"

namespace ha {

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Bounded wait for phase 0 of an mbarrier.  Returns false if the copy has not completed after the
// limit (never seen; the caller then fetches the data with ordinary loads instead).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar) {
    for (int it = 0; it < (1 << 20); ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(0u) : "memory");
        if (done) return true;
    }
    return false;
}

// z[v] += sum_k hin[v][k] * w[k][o], ascending k, one fmaf per term; the VT chains are independent
// (vector v starts at hin + v * vstride).
template <int VT>
__device__ __forceinline__ void vec_layer(const float *__restrict__ hin, const uint16_t *__restrict__ w, int ld,
                                          int o, float (&z)[VT], int vstride = kD) {
#pragma unroll 8
    for (int k = 0; k < 128; k += 4) {
        const float w0 = bf16_bits_to_float(w[(k + 0) * ld + o]);
        const float w1 = bf16_bits_to_float(w[(k + 1) * ld + o]);
        const float w2 = bf16_bits_to_float(w[(k + 2) * ld + o]);
        const float w3 = bf16_bits_to_float(w[(k + 3) * ld + o]);
        float4 hv[VT];
#pragma unroll
        for (int v = 0; v < VT; ++v) hv[v] = *reinterpret_cast<const float4 *>(hin + v * vstride + k);   // warp broadcast
#pragma unroll
        for (int v = 0; v < VT; ++v) z[v] = __fmaf_rn(hv[v].x, w0, z[v]);
#pragma unroll
        for (int v = 0; v < VT; ++v) z[v] = __fmaf_rn(hv[v].y, w1, z[v]);
#pragma unroll
        for (int v = 0; v < VT; ++v) z[v] = __fmaf_rn(hv[v].z, w2, z[v]);
#pragma unroll
        for (int v = 0; v < VT; ++v) z[v] = __fmaf_rn(hv[v].w, w3, z[v]);
    }
}

// ---- weights held transposed in shared memory: wT[o][k], so that a thread reads eight consecutive terms of
// its chain with one 16-byte load.  Against the [k][o] layout this is an eighth of the load instructions
// and half the shared-memory wavefronts, which leaves a layer bound by the latency of its fma chain.
// Rows are 256 bytes, unpadded; the 16-byte chunk c of row o is stored at position c ^ swizzle(o), which
// makes both the reads (lanes = consecutive rows, same chunk) and the transposing stores (lanes = chunks of
// one source row, i.e. rows o, o+8, ...) spread over the banks.
__device__ __forceinline__ int wt_swizzle(int o) { return (o ^ (o >> 3)) & 7; }

// Transposing fetch of a [128][kOut] bf16 matrix from global memory into wT[kOut][128] by the kThreads
// threads of the CTA, in two halves so that a caller can have the loads of several matrices in flight
// before the first store.  A warp reads whole source rows (a lane takes the same 16 bytes, eight outputs,
// of rows k and k+1) and stores the (w[k][o], w[k+1][o]) pairs as 32-bit words of row o.
template <int kThreads, int kOut>
struct TransposedFetch {
    static constexpr int kChunks = kOut / 8;            // 16-byte chunks per source row
    static constexpr int kPairs = 32 / kChunks;         // row pairs per warp instruction
    static constexpr int kUnits = 64 / kPairs, kWarps = kThreads / 32, kPer = kUnits / kWarps;
    static_assert(kUnits % kWarps == 0 && kPer >= 1, "the row pairs must split evenly over the warps");
    uint4 r0[kPer], r1[kPer];

    __device__ __forceinline__ void load(const uint16_t *__restrict__ w, int tid) {
        const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int k = 2 * ((warp * kPer + j) * kPairs + lane / kChunks), o0 = (lane % kChunks) * 8;
            r0[j] = __ldg(reinterpret_cast<const uint4 *>(w + (size_t)k * kOut + o0));
            r1[j] = __ldg(reinterpret_cast<const uint4 *>(w + (size_t)(k + 1) * kOut + o0));
        }
    }
    __device__ __forceinline__ void store(uint16_t *wT, int tid) const {
        const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int k = 2 * ((warp * kPer + j) * kPairs + lane / kChunks), ch = lane % kChunks, o0 = ch * 8;
            const uint32_t lo[4] = {r0[j].x, r0[j].y, r0[j].z, r0[j].w}, hi[4] = {r1[j].x, r1[j].y, r1[j].z, r1[j].w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int o = o0 + i, pos = ((k >> 3) ^ wt_swizzle(o)) * 8 + (k & 7);
                *reinterpret_cast<uint32_t *>(wT + o * kD + pos) = __byte_perm(lo[i >> 1], hi[i >> 1], (i & 1) ? 0x7632 : 0x5410);
            }
        }
    }
};

// z[v] += sum_k hin[v][k] * w[k][o], ascending k, one fmaf per term; wT = the transposed matrix.
template <int VT>
__device__ __forceinline__ void vec_layer_t(const float *__restrict__ hin, const uint16_t *__restrict__ wT, int o, float (&z)[VT]) {
    const uint4 *wp = reinterpret_cast<const uint4 *>(wT + o * kD);
    const int swz = wt_swizzle(o);
#pragma unroll
    for (int c = 0; c < kD / 8; ++c) {
        const uint4 wv = wp[c ^ swz];
        const uint32_t wq[4] = {wv.x, wv.y, wv.z, wv.w};
        float4 ha[VT], hb[VT];
#pragma unroll
        for (int v = 0; v < VT; ++v) {   // warp broadcasts
            ha[v] = *reinterpret_cast<const float4 *>(hin + v * kD + 8 * c);
            hb[v] = *reinterpret_cast<const float4 *>(hin + v * kD + 8 * c + 4);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float we = __uint_as_float(wq[e] << 16), wo = __uint_as_float(wq[e] & 0xffff0000u);
#pragma unroll
            for (int v = 0; v < VT; ++v) {
                const float4 &h = (e < 2) ? ha[v] : hb[v];
                z[v] = __fmaf_rn((e & 1) ? h.z : h.x, we, z[v]);
            }
#pragma unroll
            for (int v = 0; v < VT; ++v) {
                const float4 &h = (e < 2) ? ha[v] : hb[v];
                z[v] = __fmaf_rn((e & 1) ? h.w : h.y, wo, z[v]);
            }
        }
    }
}

} // namespace ha
