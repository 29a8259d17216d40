// ENCODE (Eq. 2): signature = packed sign bits of the Section 5.2 feed-forward net
// 128 -> 128 -> 128 -> 32.  Every output is one fp32 fused-multiply-add chain over ascending
// input index started from the bias, so the result does not depend on how outputs are spread
// over threads.  Two kernels: one CTA per vector for the handful of vectors of a decode step
// (latency-bound), and a token-tiled kernel with the weights held in shared memory for building
// the signature cache of a whole prompt.
#include "ha_common.cuh"

namespace ha {

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

// ------------------------------------------------------------------ decode-step kernel
//
// One CTA per (sequence, network): the G query vectors that share a network (or the one new key)
// are encoded together, so the 72 KB of weights are fetched once per CTA.  All three weight
// matrices are requested with cp.async at kernel entry (one HBM/L2 round trip instead of one per
// unrolled batch of a dependent loop); each layer starts as soon as its matrix has landed.  Thread
// o runs the fma chain of output o for every vector of the CTA (independent chains interleave).

constexpr int kVecThreads = 128;
constexpr int kVecMax = 8;   // vectors per CTA
constexpr size_t kVecSmem = (size_t)(kD * kHid + kHid * kHid + kHid * kBits) * 2 + (size_t)2 * kVecMax * kD * 4;

__device__ __forceinline__ void cp_async16_enc(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

template <int NV>
__device__ __forceinline__ void vec_layer(const float *__restrict__ hin, const uint16_t *__restrict__ w, int ld,
                                          int o, int nv, float (&z)[NV]) {
    // z[v] += sum_k hin[v][k] * w[k][o], ascending k, one fmaf per term
#pragma unroll 4
    for (int k = 0; k < 128; k += 4) {
        const float w0 = bf16_bits_to_float(w[(k + 0) * ld + o]);
        const float w1 = bf16_bits_to_float(w[(k + 1) * ld + o]);
        const float w2 = bf16_bits_to_float(w[(k + 2) * ld + o]);
        const float w3 = bf16_bits_to_float(w[(k + 3) * ld + o]);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (v < nv) {
                const float4 hv = *reinterpret_cast<const float4 *>(hin + v * kD + k);   // warp broadcast
                z[v] = __fmaf_rn(hv.x, w0, z[v]);
                z[v] = __fmaf_rn(hv.y, w1, z[v]);
                z[v] = __fmaf_rn(hv.z, w2, z[v]);
                z[v] = __fmaf_rn(hv.w, w3, z[v]);
            }
        }
    }
}

template <int NV>
__global__ void __launch_bounds__(kVecThreads) encode_vec_kernel(EncodeJob ja, EncodeJob jb) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint16_t *sw1 = reinterpret_cast<uint16_t *>(smem);
    uint16_t *sw2 = sw1 + kD * kHid;
    uint16_t *sw3 = sw2 + kHid * kHid;
    float *actA = reinterpret_cast<float *>(sw3 + kHid * kBits);   // [NV][128]
    float *actB = actA + kVecMax * kD;

    int i = blockIdx.x;
    const bool second = i >= ja.n_cta;
    const EncodeJob &J = second ? jb : ja;
    if (second) i -= ja.n_cta;
    const int n_nets = J.n_heads / J.heads_per_kv;
    const int b = i / n_nets, net = i % n_nets;
    const int nv = J.heads_per_kv;   // <= NV
    const int o = threadIdx.x;

    // ---- request all weights (three commit groups), then the inputs
    {
        const unsigned char *g1 = reinterpret_cast<const unsigned char *>(J.map.w1 + (size_t)net * kD * kHid);
        const unsigned char *g2 = reinterpret_cast<const unsigned char *>(J.map.w2 + (size_t)net * kHid * kHid);
        const unsigned char *g3 = reinterpret_cast<const unsigned char *>(J.map.w3 + (size_t)net * kHid * kBits);
        const uint32_t s1 = (uint32_t)__cvta_generic_to_shared(sw1), s2 = (uint32_t)__cvta_generic_to_shared(sw2),
                       s3 = (uint32_t)__cvta_generic_to_shared(sw3);
        for (int c = o; c < kD * kHid / 8; c += kVecThreads) cp_async16_enc(s1 + c * 16, g1 + c * 16);
        asm volatile("cp.async.commit_group;" ::: "memory");
        for (int c = o; c < kHid * kHid / 8; c += kVecThreads) cp_async16_enc(s2 + c * 16, g2 + c * 16);
        asm volatile("cp.async.commit_group;" ::: "memory");
        for (int c = o; c < kHid * kBits / 8; c += kVecThreads) cp_async16_enc(s3 + c * 16, g3 + c * 16);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const float bias1 = J.map.b1 ? __ldg(J.map.b1 + net * kHid + o) : 0.0f;
    const float bias2 = J.map.b2 ? __ldg(J.map.b2 + net * kHid + o) : 0.0f;
    const float bias3 = (J.map.b3 && o < kBits) ? __ldg(J.map.b3 + net * kBits + o) : 0.0f;
    // the weights do not depend on earlier kernels of the stream; the vectors to encode may
    pdl_launch_dependents();
    pdl_wait();
    for (int v = 0; v < nv; ++v) {
        const uint16_t *x = J.x + (long long)b * J.x_sb + (long long)(net * J.heads_per_kv + v) * J.x_sh;
        actA[v * kD + o] = bf16_bits_to_float(__ldg(x + o));
    }

    int slot = 0;
    if (J.slot) slot = J.slot[b] - J.slot_minus_one;   // a negative slot skips the sequence (no write below)

    float z[NV];
    // ---- layer 1
    asm volatile("cp.async.wait_group 2;" ::: "memory");
    __syncthreads();
#pragma unroll
    for (int v = 0; v < NV; ++v) z[v] = bias1;
    vec_layer<NV>(actA, sw1, kHid, o, nv, z);
#pragma unroll
    for (int v = 0; v < NV; ++v)
        if (v < nv) actB[v * kD + o] = (z[v] > 0.0f) ? z[v] : 0.0f;
    // ---- layer 2
    asm volatile("cp.async.wait_group 1;" ::: "memory");
    __syncthreads();
#pragma unroll
    for (int v = 0; v < NV; ++v) z[v] = bias2;
    vec_layer<NV>(actB, sw2, kHid, o, nv, z);
    // actA was last read in layer 1, which every thread left before the barrier above
#pragma unroll
    for (int v = 0; v < NV; ++v)
        if (v < nv) actA[v * kD + o] = (z[v] > 0.0f) ? z[v] : 0.0f;
    // ---- layer 3: one output bit per lane of warp 0
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if (o < kBits) {
#pragma unroll
        for (int v = 0; v < NV; ++v) z[v] = bias3;
        vec_layer<NV>(actA, sw3, kBits, o, nv, z);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const uint32_t code = __ballot_sync(0xffffffffu, z[v] > 0.0f);
            if (o == 0 && v < nv && slot >= 0)
                J.codes[(long long)b * J.c_sb + (long long)(net * J.heads_per_kv + v) * J.c_sh + slot] = code;
        }
    }
}

template <int NV>
static cudaError_t launch_vec_t(const EncodeJob &a, const EncodeJob &b, cudaStream_t st) {
    static bool done[64] = {};   // opt in to > 48 KB of shared memory once per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(encode_vec_kernel<NV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kVecSmem);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    cudaError_t e = launch_pdl(encode_vec_kernel<NV>, dim3(a.n_cta + b.n_cta), dim3(kVecThreads), kVecSmem, st, a, b);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_encode_vectors(const EncodeJob &a, const EncodeJob &b, cudaStream_t st) {
    if (a.n_cta + b.n_cta <= 0) return cudaSuccess;
    const int nv = max(a.n_cta > 0 ? a.heads_per_kv : 1, b.n_cta > 0 ? b.heads_per_kv : 1);
    if (nv <= 1) return launch_vec_t<1>(a, b, st);
    if (nv <= 2) return launch_vec_t<2>(a, b, st);
    if (nv <= 4) return launch_vec_t<4>(a, b, st);
    if (nv <= 8) return launch_vec_t<8>(a, b, st);
    return cudaErrorInvalidValue;
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
