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

// z[v] += sum_k hin[v][k] * w[k][o], ascending k, one fmaf per term; the VT chains are independent.
template <int VT>
__device__ __forceinline__ void vec_layer(const float *__restrict__ hin, const uint16_t *__restrict__ w, int ld,
                                          int o, float (&z)[VT]) {
#pragma unroll 8
    for (int k = 0; k < 128; k += 4) {
        const float w0 = bf16_bits_to_float(w[(k + 0) * ld + o]);
        const float w1 = bf16_bits_to_float(w[(k + 1) * ld + o]);
        const float w2 = bf16_bits_to_float(w[(k + 2) * ld + o]);
        const float w3 = bf16_bits_to_float(w[(k + 3) * ld + o]);
        float4 hv[VT];
#pragma unroll
        for (int v = 0; v < VT; ++v) hv[v] = *reinterpret_cast<const float4 *>(hin + v * kD + k);   // warp broadcast
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

} // namespace ha
