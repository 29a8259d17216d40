// ENCODE (Eq. 2): signature = packed sign bits of the Section 5.2 feed-forward net
// 128 -> 128 -> 128 -> 32.  Every output is one fp32 fused-multiply-add chain over ascending
// input index started from the bias, so the result does not depend on how outputs are spread
// over threads.  Two kernels: one CTA per vector for the handful of vectors of a decode step
// (latency-bound), and a token-tiled kernel with the weights held in shared memory for building
// the signature cache of a whole prompt.
#include "ha_common.cuh"

namespace ha {

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

// ------------------------------------------------------------------ per-vector kernel

__device__ __forceinline__ float dense_chain_128(const float *h, const uint16_t *__restrict__ w, int ld,
                                                 float z) {
    // z += sum_k h[k] * w[k*ld], ascending k, one fmaf per term
#pragma unroll 32
    for (int k = 0; k < 128; ++k) z = __fmaf_rn(h[k], bf16_bits_to_float(__ldg(w + (size_t)k * ld)), z);
    return z;
}

__global__ void __launch_bounds__(128) encode_vec_kernel(EncodeJob ja, EncodeJob jb) {
    __shared__ float h0[kD];
    __shared__ float h1[kHid];
    int v = blockIdx.x;
    const EncodeJob &J = (v < ja.n_vec) ? ja : jb;
    if (v >= ja.n_vec) v -= ja.n_vec;
    const int b = v / J.n_heads, h = v % J.n_heads;
    const int net = h / J.heads_per_kv;
    const int o = threadIdx.x;

    int slot = 0;
    if (J.slot) {
        slot = J.slot[b] - J.slot_minus_one;
        if (slot < 0) return;
    }
    const uint16_t *x = J.x + (long long)b * J.x_sb + (long long)h * J.x_sh;
    h0[o] = bf16_bits_to_float(x[o]);
    __syncthreads();

    float z = J.map.b1 ? J.map.b1[net * kHid + o] : 0.0f;
    z = dense_chain_128(h0, J.map.w1 + (size_t)net * kD * kHid + o, kHid, z);
    h1[o] = (z > 0.0f) ? z : 0.0f;
    __syncthreads();

    z = J.map.b2 ? J.map.b2[net * kHid + o] : 0.0f;
    z = dense_chain_128(h1, J.map.w2 + (size_t)net * kHid * kHid + o, kHid, z);
    h0[o] = (z > 0.0f) ? z : 0.0f;
    __syncthreads();

    if (o < kBits) {   // warp 0: one output bit per lane
        z = J.map.b3 ? J.map.b3[net * kBits + o] : 0.0f;
        z = dense_chain_128(h0, J.map.w3 + (size_t)net * kHid * kBits + o, kBits, z);
        const uint32_t code = __ballot_sync(0xffffffffu, z > 0.0f);
        if (o == 0) J.codes[(long long)b * J.c_sb + (long long)h * J.c_sh + slot] = code;
    }
}

cudaError_t launch_encode_vectors(const EncodeJob &a, const EncodeJob &b, cudaStream_t st) {
    const int n = a.n_vec + b.n_vec;
    if (n <= 0) return cudaSuccess;
    encode_vec_kernel<<<n, 128, 0, st>>>(a, b);
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ token-tiled bulk kernel

constexpr int kTile = 64;             // tokens per CTA
constexpr int kBulkThreads = 256;
constexpr int kActLd = kD + 4;        // padded row of the activation tile (floats)
constexpr size_t kBulkSmem = (size_t)(kD * kHid + kHid * kHid + kHid * kBits) * 2   // bf16 weights
                             + (size_t)2 * kTile * kActLd * 4;                    // two activation tiles

// One hidden layer for a 64-token tile: thread (o, half) owns output o of 32 tokens.
__device__ __forceinline__ void bulk_hidden_layer(const float *__restrict__ in, float *__restrict__ out,
                                                  const uint16_t *__restrict__ w, const float *bias, int o,
                                                  int half) {
    float z[32];
    const float b = bias ? bias[o] : 0.0f;
#pragma unroll
    for (int t = 0; t < 32; ++t) z[t] = b;
    const float *hin = in + (size_t)half * 32 * kActLd;
    for (int k = 0; k < 128; k += 4) {
        const float w0 = bf16_bits_to_float(w[(k + 0) * kHid + o]);
        const float w1 = bf16_bits_to_float(w[(k + 1) * kHid + o]);
        const float w2 = bf16_bits_to_float(w[(k + 2) * kHid + o]);
        const float w3 = bf16_bits_to_float(w[(k + 3) * kHid + o]);
#pragma unroll
        for (int t = 0; t < 32; ++t) {
            const float4 hv = *reinterpret_cast<const float4 *>(hin + t * kActLd + k);   // warp broadcast
            z[t] = __fmaf_rn(hv.x, w0, z[t]);
            z[t] = __fmaf_rn(hv.y, w1, z[t]);
            z[t] = __fmaf_rn(hv.z, w2, z[t]);
            z[t] = __fmaf_rn(hv.w, w3, z[t]);
        }
    }
    float *hout = out + (size_t)half * 32 * kActLd;
#pragma unroll
    for (int t = 0; t < 32; ++t) hout[t * kActLd + o] = (z[t] > 0.0f) ? z[t] : 0.0f;
}

__global__ void __launch_bounds__(kBulkThreads) encode_bulk_kernel(MapView map, int heads_per_kv, TensorView x,
                                                                  int T, uint32_t *codes, long long c_sb,
                                                                  long long c_sh) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint16_t *sw1 = reinterpret_cast<uint16_t *>(smem);
    uint16_t *sw2 = sw1 + kD * kHid;
    uint16_t *sw3 = sw2 + kHid * kHid;
    float *actA = reinterpret_cast<float *>(sw3 + kHid * kBits);
    float *actB = actA + kTile * kActLd;

    const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int net = h / heads_per_kv;
    const int tid = threadIdx.x;
    const int t0 = tile * kTile;
    const int nt = min(kTile, T - t0);

    // weights of this head's network -> shared memory (16-byte copies)
    {
        const uint4 *g1 = reinterpret_cast<const uint4 *>(map.w1 + (size_t)net * kD * kHid);
        const uint4 *g2 = reinterpret_cast<const uint4 *>(map.w2 + (size_t)net * kHid * kHid);
        const uint4 *g3 = reinterpret_cast<const uint4 *>(map.w3 + (size_t)net * kHid * kBits);
        uint4 *s1 = reinterpret_cast<uint4 *>(sw1), *s2 = reinterpret_cast<uint4 *>(sw2), *s3 = reinterpret_cast<uint4 *>(sw3);
        for (int i = tid; i < kD * kHid / 8; i += kBulkThreads) s1[i] = __ldg(g1 + i);
        for (int i = tid; i < kHid * kHid / 8; i += kBulkThreads) s2[i] = __ldg(g2 + i);
        for (int i = tid; i < kHid * kBits / 8; i += kBulkThreads) s3[i] = __ldg(g3 + i);
    }
    // input tile -> fp32 (rows beyond the sequence are zero; their codes are not written)
    const uint16_t *xb = x.ptr + (long long)b * x.sb + (long long)h * x.sh;
    for (int i = tid; i < kTile * (kD / 8); i += kBulkThreads) {
        const int t = i / (kD / 8), c = i % (kD / 8);
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (t < nt) raw = __ldg(reinterpret_cast<const uint4 *>(xb + (long long)(t0 + t) * x.sn) + c);
        const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
        float *dst = actA + t * kActLd + c * 8;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            dst[2 * e] = __uint_as_float(r[e] << 16);
            dst[2 * e + 1] = __uint_as_float(r[e] & 0xffff0000u);
        }
    }
    __syncthreads();

    const int o = tid & 127, half = tid >> 7;
    bulk_hidden_layer(actA, actB, sw1, map.b1 ? map.b1 + net * kHid : nullptr, o, half);
    __syncthreads();
    bulk_hidden_layer(actB, actA, sw2, map.b2 ? map.b2 + net * kHid : nullptr, o, half);
    __syncthreads();

    // last layer: lane = output bit, warp w owns tokens 8w .. 8w+7
    {
        const int lane = tid & 31, w = tid >> 5;
        float z[8];
        const float bb = map.b3 ? map.b3[net * kBits + lane] : 0.0f;
#pragma unroll
        for (int t = 0; t < 8; ++t) z[t] = bb;
        const float *hin = actA + (size_t)w * 8 * kActLd;
        for (int k = 0; k < 128; k += 4) {
            const float w0 = bf16_bits_to_float(sw3[(k + 0) * kBits + lane]);
            const float w1 = bf16_bits_to_float(sw3[(k + 1) * kBits + lane]);
            const float w2 = bf16_bits_to_float(sw3[(k + 2) * kBits + lane]);
            const float w3 = bf16_bits_to_float(sw3[(k + 3) * kBits + lane]);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const float4 hv = *reinterpret_cast<const float4 *>(hin + t * kActLd + k);
                z[t] = __fmaf_rn(hv.x, w0, z[t]);
                z[t] = __fmaf_rn(hv.y, w1, z[t]);
                z[t] = __fmaf_rn(hv.z, w2, z[t]);
                z[t] = __fmaf_rn(hv.w, w3, z[t]);
            }
        }
        uint32_t *cb = codes + (long long)b * c_sb + (long long)h * c_sh + t0;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint32_t code = __ballot_sync(0xffffffffu, z[t] > 0.0f);
            if (lane == 0 && w * 8 + t < nt) cb[w * 8 + t] = code;
        }
    }
}

cudaError_t launch_encode_bulk(const MapView &map, int heads_per_kv, TensorView x, int B, int H, int T,
                               uint32_t *codes, long long c_sb, long long c_sh, cudaStream_t st) {
    // the attribute belongs to the current device; setting it per call keeps multi-device processes right
    cudaError_t e = cudaFuncSetAttribute(encode_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kBulkSmem);
    if (e != cudaSuccess) return e;
    dim3 grid((T + kTile - 1) / kTile, H, B);
    encode_bulk_kernel<<<grid, kBulkThreads, kBulkSmem, st>>>(map, heads_per_kv, x, T, codes, c_sb, c_sh);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha
