// ENCODE (Eq. 2): signature = packed sign bits of the Section 5.2 feed-forward net
// 128 -> 128 -> 128 -> 32.  Every output is one fp32 fused-multiply-add chain over ascending
// input index started from the bias, so the result does not depend on how outputs are spread
// over threads.  Two kernels: one for the handful of vectors of a decode step (latency-bound), and a
// token-tiled kernel with the weights held in shared memory for building
// the signature cache of a whole prompt.
#include "ha_encode_dev.cuh"

namespace ha {


// ------------------------------------------------------------------ decode-step kernel
//
// The vectors of one network (the queries of a KV head over the whole batch, or the appended keys)
// are cut into items of NV vectors.  A CTA belongs to one network, fetches its 72 KB of weights
// once and encodes the items part, part + P, ... of that network.  A step of few vectors uses
// NV = 1 and one item per CTA (the chains of different vectors run on different SMs); a larger one
// as many vectors per CTA as it takes for all CTAs to be resident at once, in items of up to 8
// vectors (launch_encode_vectors), so that neither a second wave nor the weight traffic grows the latency.
// One thread requests the three weight matrices with bulk asynchronous copies (TMA, one mbarrier
// per matrix) at kernel entry, before the programmatic-launch wait: the fetch overlaps the
// preceding kernels and costs no issue slots; each layer starts as soon as its matrix has landed.
// Thread o runs the fma chains of output o for every vector of the item.  The layers are bound by
// shared-memory bandwidth (one 2-byte weight per lane and term), so one warp per scheduler that
// reuses each weight for all its vectors beats more warps that each re-read the matrix.

constexpr int kVecThreads = 128;
constexpr size_t kVecWeightBytes = (size_t)(kD * kHid + kHid * kHid + kHid * kBits) * 2;

template <int NV>
__global__ void __launch_bounds__(kVecThreads) encode_vec_kernel(EncodeJob ja, EncodeJob jb) {
    extern __shared__ __align__(128) unsigned char vec_smem[];
    __shared__ __align__(8) unsigned long long s_bar[3];
    uint16_t *sw1 = reinterpret_cast<uint16_t *>(vec_smem);
    uint16_t *sw2 = sw1 + kD * kHid;
    uint16_t *sw3 = sw2 + kHid * kHid;
    float *actA = reinterpret_cast<float *>(sw3 + kHid * kBits);   // [NV][128]
    float *actB = actA + NV * kD;

    int i = blockIdx.x;
    const bool second = i >= ja.n_cta;
    const EncodeJob &J = second ? jb : ja;
    if (second) i -= ja.n_cta;
    const int P = J.cta_per_net, net = i / P, part = i % P;
    const int hpk = J.heads_per_kv;
    const int n_vec = J.batch * hpk;                 // vectors of this network: t -> (b = t / hpk, head net*hpk + t % hpk)
    const int n_items = (n_vec + NV - 1) / NV;
    const int tid = threadIdx.x, o = tid;

    const uint16_t *g1 = J.map.w1 + (size_t)net * kD * kHid;
    const uint16_t *g2 = J.map.w2 + (size_t)net * kHid * kHid;
    const uint16_t *g3 = J.map.w3 + (size_t)net * kHid * kBits;
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(&s_bar[0]);
    // ---- request all weights: three bulk copies, one mbarrier each
    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        mbar_init(bar0 + 16, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar0, kD * kHid * 2);
        bulk_g2s((uint32_t)__cvta_generic_to_shared(sw1), g1, kD * kHid * 2, bar0);
        mbar_expect_tx(bar0 + 8, kHid * kHid * 2);
        bulk_g2s((uint32_t)__cvta_generic_to_shared(sw2), g2, kHid * kHid * 2, bar0 + 8);
        mbar_expect_tx(bar0 + 16, kHid * kBits * 2);
        bulk_g2s((uint32_t)__cvta_generic_to_shared(sw3), g3, kHid * kBits * 2, bar0 + 16);
    }
    const float bias1 = J.map.b1 ? __ldg(J.map.b1 + net * kHid + o) : 0.0f;
    const float bias2 = J.map.b2 ? __ldg(J.map.b2 + net * kHid + o) : 0.0f;
    const float bias3 = J.map.b3 ? __ldg(J.map.b3 + net * kBits + (tid & (kBits - 1))) : 0.0f;
    // The weights do not depend on earlier kernels of the stream; the vectors to encode may.  The
    // kernels behind this one are released only after the wait: whatever they read before their own
    // wait (sequence lengths, budgets, signatures) is then final, whoever wrote it earlier in the stream.
    pdl_wait();
    pdl_launch_dependents();

    // wait for one weight matrix; if the bulk copy never reports completion, load it the ordinary way
    // (the decision is taken by the whole CTA together, so that the barrier below is never divergent)
    auto weights_ready = [&](int which, uint16_t *dst, const uint16_t *src, int n_elems) {
        const bool ok = mbar_wait_bounded(bar0 + 8 * which);
        if (__syncthreads_or(!ok)) {
            for (int c = tid; c < n_elems / 8; c += kVecThreads)
                reinterpret_cast<uint4 *>(dst)[c] = __ldg(reinterpret_cast<const uint4 *>(src) + c);
            __syncthreads();
        }
    };

    bool first = true;
    for (int item = part; item < n_items; item += P) {   // CTA-uniform
        const int t0 = item * NV, nv = min(NV, n_vec - t0);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float xv = 0.0f;   // unused slots are zero rows (their chains are computed and dropped)
            if (v < nv) {
                const int t = t0 + v;
                const uint16_t *x = J.x + (long long)(t / hpk) * J.x_sb + (long long)(net * hpk + t % hpk) * J.x_sh;
                xv = bf16_bits_to_float(__ldg(x + o));
            }
            actA[v * kD + o] = xv;
        }
        __syncthreads();   // mbarrier inits and the inputs are visible to every thread

        float z[NV];
        // ---- layer 1
        if (first) weights_ready(0, sw1, g1, kD * kHid);
#pragma unroll
        for (int v = 0; v < NV; ++v) z[v] = bias1;
        vec_layer<NV>(actA, sw1, kHid, o, z);
#pragma unroll
        for (int v = 0; v < NV; ++v) actB[v * kD + o] = (z[v] > 0.0f) ? z[v] : 0.0f;
        __syncthreads();
        // ---- layer 2
        if (first) weights_ready(1, sw2, g2, kHid * kHid);
#pragma unroll
        for (int v = 0; v < NV; ++v) z[v] = bias2;
        vec_layer<NV>(actB, sw2, kHid, o, z);
        // actA was last read in layer 1, which every thread left before the barrier above
#pragma unroll
        for (int v = 0; v < NV; ++v) actA[v * kD + o] = (z[v] > 0.0f) ? z[v] : 0.0f;
        __syncthreads();
        // ---- layer 3: one output bit per lane; warp w takes vectors w, w + 4 (their chains interleaved)
        if (first) weights_ready(2, sw3, g3, kHid * kBits);
        first = false;
        {
            constexpr int kWarps = kVecThreads / 32, VT3 = (NV + kWarps - 1) / kWarps;
            const int warp = tid >> 5, lane = tid & 31;
            if (warp < nv) {   // warp-uniform; chains of slots >= nv read rows of the activation buffers and are dropped
                float z3[VT3];
#pragma unroll
                for (int i = 0; i < VT3; ++i) z3[i] = bias3;
                vec_layer<VT3>(actA + warp * kD, sw3, kBits, lane, z3, kWarps * kD);
#pragma unroll
                for (int i = 0; i < VT3; ++i) {
                    const int v = warp + i * kWarps;
                    const uint32_t code = __ballot_sync(0xffffffffu, z3[i] > 0.0f);
                    if (v < nv) {
                        const int t = t0 + v, b = t / hpk;
                        int slot = 0;
                        if (J.slot) slot = J.slot[b] - J.slot_minus_one;   // a negative slot skips the sequence
                        if (lane == 0 && slot >= 0)
                            *encode_slot_ptr(J, b, net * hpk + t % hpk, slot) = code;
                    }
                }
            }
        }
        __syncthreads();   // layer 3 has read actA before the next item overwrites it
    }
}

template <int NV>
static cudaError_t launch_vec_t(const EncodeJob &a, const EncodeJob &b, cudaStream_t st) {
    constexpr size_t smem = kVecWeightBytes + (size_t)2 * NV * kD * 4;
    static bool done[64] = {};   // opt in to > 48 KB of shared memory once per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(encode_vec_kernel<NV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    cudaError_t e = launch_pdl(encode_vec_kernel<NV>, dim3(a.n_cta + b.n_cta), dim3(kVecThreads), smem, st, a, b);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ decode-step kernel for large batches
//
// From a few hundred vectors per step on, one output per thread wastes the shared-memory port: every weight is a
// 2-byte load that serves a single fma chain per vector.  Here a CTA of 64 NG threads encodes a TILE of NG x VPT
// vectors of one network with register tiling: a thread owns two neighbouring outputs of VPT
// vectors, so a 4-byte weight load feeds 2 VPT chains and a 16-byte activation load (a warp-wide broadcast) feeds
// four terms of two chains.  Chains stay what Eq. 2's network is defined as here: one fused multiply-add per term,
// ascending input index, started from the bias; only their distribution over threads changes, so the signatures
// are bit-identical to encode_vec_kernel's.  Weights arrive by the same three bulk copies, requested before the
// programmatic-launch wait.
constexpr int kTileMinVectors = 40;   // vectors per network (both sides together) from which the tiled kernel takes the step
constexpr int kTileActLd = kD + 4;   // padded activation row (floats)

template <int VPT, int NG>
__global__ void __launch_bounds__(64 * NG) encode_tile_kernel(EncodeJob ja, EncodeJob jb) {
    constexpr int TV = NG * VPT;   // vectors per tile: NG vector groups (64 threads each) x VPT
    constexpr int kTileThreads = 64 * NG;
    extern __shared__ __align__(128) unsigned char tile_smem[];
    __shared__ __align__(8) unsigned long long s_bar[3];
    uint16_t *sw1 = reinterpret_cast<uint16_t *>(tile_smem);
    uint16_t *sw2 = sw1 + kD * kHid;
    uint16_t *sw3 = sw2 + kHid * kHid;
    float *actA = reinterpret_cast<float *>(sw3 + kHid * kBits);   // [TV][kTileActLd]
    float *actB = actA + TV * kTileActLd;

    int i = blockIdx.x;
    const bool second = i >= ja.n_cta;
    const EncodeJob &J = second ? jb : ja;
    if (second) i -= ja.n_cta;
    const int tiles_per_net = J.cta_per_net, net = i / tiles_per_net, tile = i % tiles_per_net;
    const int hpk = J.heads_per_kv;
    const int n_vec = J.batch * hpk;   // vectors of this network: t -> (b = t / hpk, head net*hpk + t % hpk)
    const int t0 = tile * TV, nv = min(TV, n_vec - t0);
    const int tid = threadIdx.x;

    const uint16_t *g1 = J.map.w1 + (size_t)net * kD * kHid;
    const uint16_t *g2 = J.map.w2 + (size_t)net * kHid * kHid;
    const uint16_t *g3 = J.map.w3 + (size_t)net * kHid * kBits;
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(&s_bar[0]);
    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        mbar_init(bar0 + 16, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar0, kD * kHid * 2);
        bulk_g2s((uint32_t)__cvta_generic_to_shared(sw1), g1, kD * kHid * 2, bar0);
        mbar_expect_tx(bar0 + 8, kHid * kHid * 2);
        bulk_g2s((uint32_t)__cvta_generic_to_shared(sw2), g2, kHid * kHid * 2, bar0 + 8);
        mbar_expect_tx(bar0 + 16, kHid * kBits * 2);
        bulk_g2s((uint32_t)__cvta_generic_to_shared(sw3), g3, kHid * kBits * 2, bar0 + 16);
    }
    // hidden layers: thread = (output pair op, vector group vg); last layer: thread = (output pair op3, vector v3)
    const int op = tid & 63, vg = tid >> 6;
    float b1[2], b2[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        b1[e] = J.map.b1 ? __ldg(J.map.b1 + net * kHid + 2 * op + e) : 0.0f;
        b2[e] = J.map.b2 ? __ldg(J.map.b2 + net * kHid + 2 * op + e) : 0.0f;
    }
    pdl_wait();                 // the vectors may come from the kernel in front; the weights do not
    pdl_launch_dependents();

    // the tile's vectors -> fp32 rows (slots past the batch are zero rows; their signatures are dropped)
    for (int e = tid; e < TV * (kD / 8); e += kTileThreads) {
        const int v = e / (kD / 8), c = e % (kD / 8);
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (v < nv) {
            const int t = t0 + v;
            const uint16_t *x = J.x + (long long)(t / hpk) * J.x_sb + (long long)(net * hpk + t % hpk) * J.x_sh;
            raw = __ldg(reinterpret_cast<const uint4 *>(x) + c);
        }
        const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
        float *dst = actA + v * kTileActLd + c * 8;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            dst[2 * q] = __uint_as_float(r[q] << 16);
            dst[2 * q + 1] = __uint_as_float(r[q] & 0xffff0000u);
        }
    }
    __syncthreads();   // inputs and mbarrier inits visible

    auto weights_ready = [&](int which, uint16_t *dst, const uint16_t *src, int n_elems) {
        const bool ok = mbar_wait_bounded(bar0 + 8 * which);
        if (__syncthreads_or(!ok)) {   // never seen: fetch the matrix with ordinary loads instead
            for (int c = tid; c < n_elems / 8; c += kTileThreads)
                reinterpret_cast<uint4 *>(dst)[c] = __ldg(reinterpret_cast<const uint4 *>(src) + c);
            __syncthreads();
        }
    };
    // one hidden layer: out[v][2 op + e] = relu(bias[e] + sum_k in[v][k] w[k][2 op + e]) for the VPT vectors of group vg
    auto hidden = [&](const float *in, float *out, const uint16_t *w, const float (&bias)[2]) {
        float z[VPT][2];
#pragma unroll
        for (int v = 0; v < VPT; ++v) { z[v][0] = bias[0]; z[v][1] = bias[1]; }
        const float *hin = in + (size_t)vg * VPT * kTileActLd;
#pragma unroll 4
        for (int k = 0; k < 128; k += 4) {
            float wf[4][2];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const uint32_t wv = *reinterpret_cast<const uint32_t *>(w + (k + t) * kHid + 2 * op);
                wf[t][0] = __uint_as_float(wv << 16);
                wf[t][1] = __uint_as_float(wv & 0xffff0000u);
            }
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                const float4 hv = *reinterpret_cast<const float4 *>(hin + v * kTileActLd + k);   // warp broadcast
#pragma unroll
                for (int e = 0; e < 2; ++e) {   // ascending term index within every chain
                    z[v][e] = __fmaf_rn(hv.x, wf[0][e], z[v][e]);
                    z[v][e] = __fmaf_rn(hv.y, wf[1][e], z[v][e]);
                    z[v][e] = __fmaf_rn(hv.z, wf[2][e], z[v][e]);
                    z[v][e] = __fmaf_rn(hv.w, wf[3][e], z[v][e]);
                }
            }
        }
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float2 r;
            r.x = (z[v][0] > 0.0f) ? z[v][0] : 0.0f;
            r.y = (z[v][1] > 0.0f) ? z[v][1] : 0.0f;
            *reinterpret_cast<float2 *>(out + (size_t)(vg * VPT + v) * kTileActLd + 2 * op) = r;
        }
    };
    weights_ready(0, sw1, g1, kD * kHid);
    hidden(actA, actB, sw1, b1);
    __syncthreads();
    weights_ready(1, sw2, g2, kHid * kHid);
    hidden(actB, actA, sw2, b2);
    __syncthreads();
    weights_ready(2, sw3, g3, kHid * kBits);
    // last layer, 32 outputs: thread (op3 = output pair, v3 = vector); a half-warp holds the 16 pairs of one vector
    {
        const int lane = tid & 31, op3 = tid & 15, v3 = tid >> 4;
        if (v3 < TV) {   // warp-uniform (TV is 4, 8 or 16; the CTA has at least 16 TV threads)
            float z0 = J.map.b3 ? __ldg(J.map.b3 + net * kBits + 2 * op3) : 0.0f;
            float z1 = J.map.b3 ? __ldg(J.map.b3 + net * kBits + 2 * op3 + 1) : 0.0f;
            const float *hin = actA + (size_t)v3 * kTileActLd;
#pragma unroll 4
            for (int k = 0; k < 128; k += 4) {
                const float4 hv = *reinterpret_cast<const float4 *>(hin + k);
                float wf[4][2];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const uint32_t wv = *reinterpret_cast<const uint32_t *>(sw3 + (k + t) * kBits + 2 * op3);
                    wf[t][0] = __uint_as_float(wv << 16);
                    wf[t][1] = __uint_as_float(wv & 0xffff0000u);
                }
                z0 = __fmaf_rn(hv.x, wf[0][0], z0); z1 = __fmaf_rn(hv.x, wf[0][1], z1);
                z0 = __fmaf_rn(hv.y, wf[1][0], z0); z1 = __fmaf_rn(hv.y, wf[1][1], z1);
                z0 = __fmaf_rn(hv.z, wf[2][0], z0); z1 = __fmaf_rn(hv.z, wf[2][1], z1);
                z0 = __fmaf_rn(hv.w, wf[3][0], z0); z1 = __fmaf_rn(hv.w, wf[3][1], z1);
            }
            const uint32_t even = __ballot_sync(0xffffffffu, z0 > 0.0f), odd = __ballot_sync(0xffffffffu, z1 > 0.0f);
            auto spread16 = [](uint32_t v) {   // bit i -> bit 2 i
                v = (v | (v << 8)) & 0x00ff00ffu;
                v = (v | (v << 4)) & 0x0f0f0f0fu;
                v = (v | (v << 2)) & 0x33333333u;
                v = (v | (v << 1)) & 0x55555555u;
                return v;
            };
            const int shift = lane & 16;   // this half-warp's 16 bits of either ballot
            const uint32_t code = spread16((even >> shift) & 0xffffu) | (spread16((odd >> shift) & 0xffffu) << 1);
            if (op3 == 0 && v3 < nv) {
                const int t = t0 + v3, b = t / hpk;
                int slot = 0;
                if (J.slot) slot = J.slot[b] - J.slot_minus_one;   // a negative slot skips the sequence
                if (slot >= 0) *encode_slot_ptr(J, b, net * hpk + t % hpk, slot) = code;
            }
        }
    }
}

template <int VPT, int NG>
static cudaError_t launch_tile_t(const EncodeJob &a, const EncodeJob &b, cudaStream_t st) {
    static_assert(64 * NG >= 16 * NG * VPT, "the last layer needs 16 threads per vector");
    constexpr size_t smem = kVecWeightBytes + (size_t)2 * NG * VPT * kTileActLd * 4;
    static bool done[64] = {};   // opt in to > 48 KB of shared memory once per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(encode_tile_kernel<VPT, NG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    cudaError_t e = launch_pdl(encode_tile_kernel<VPT, NG>, dim3(a.n_cta + b.n_cta), dim3(64 * NG), smem, st, a, b);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

// `a` and `b` arrive with n_cta = the number of (sequence, network) pairs (0 = no such job); the item
// width and the CTAs per network are chosen here: the smallest number m of vectors per CTA for which
// all CTAs are resident at once (two CTAs of 76 KB fit one SM; a second wave would double the latency),
// each network getting CTAs in proportion to its vectors, and a CTA's m vectors cut into the fewest
// items of at most 8 vectors, equal in width.
cudaError_t launch_encode_vectors(const EncodeJob &a_in, const EncodeJob &b_in, cudaStream_t st) {
    if (a_in.n_cta + b_in.n_cta <= 0) return cudaSuccess;
    EncodeJob job[2] = {a_in, b_in};
    int nets[2], vec_per_net[2];
    for (int j = 0; j < 2; ++j) {
        EncodeJob &J = job[j];
        nets[j] = (J.n_cta > 0) ? J.n_heads / J.heads_per_kv : 0;
        J.batch = (J.n_cta > 0) ? J.n_cta / nets[j] : 0;
        vec_per_net[j] = J.batch * J.heads_per_kv;
    }
    const long long room = 2LL * sm_count();
    if (vec_per_net[0] + vec_per_net[1] >= kTileMinVectors) {
        // large batch: tiles of 4, 8 or 16 vectors per CTA, the smallest for which all CTAs are resident at once
        int tv = 4;
        auto tiles = [&](int t) {
            long long n = 0;
            for (int j = 0; j < 2; ++j) n += (long long)nets[j] * ((vec_per_net[j] + t - 1) / t);
            return n;
        };
        while (tv < 16 && tiles(tv) > room) tv *= 2;
        for (int j = 0; j < 2; ++j) {
            EncodeJob &J = job[j];
            J.cta_per_net = (vec_per_net[j] + tv - 1) / tv;   // tiles per network
            J.n_cta = nets[j] * J.cta_per_net;
        }
        if (tv == 4) return launch_tile_t<1, 4>(job[0], job[1], st);
        if (tv == 8) return launch_tile_t<2, 4>(job[0], job[1], st);
        return launch_tile_t<4, 4>(job[0], job[1], st);
    }
    auto ctas = [&](int m) {
        long long n = 0;
        for (int j = 0; j < 2; ++j) n += (long long)nets[j] * ((vec_per_net[j] + m - 1) / m);
        return n;
    };
    const int m_max = vec_per_net[0] > vec_per_net[1] ? vec_per_net[0] : vec_per_net[1];   // one CTA per network
    int m = 1;
    while (m < m_max && ctas(m) > room) ++m;   // more networks than CTA slots: several waves, nothing to balance
    const int items_per_cta = (m + 7) / 8, nv = (m + items_per_cta - 1) / items_per_cta;
    for (int j = 0; j < 2; ++j) {
        EncodeJob &J = job[j];
        J.cta_per_net = (vec_per_net[j] + m - 1) / m;
        J.n_cta = nets[j] * J.cta_per_net;
    }
    switch (nv) {
        case 1: return launch_vec_t<1>(job[0], job[1], st);
        case 2: return launch_vec_t<2>(job[0], job[1], st);
        case 3: return launch_vec_t<3>(job[0], job[1], st);
        case 4: return launch_vec_t<4>(job[0], job[1], st);
        case 5: return launch_vec_t<5>(job[0], job[1], st);
        case 6: return launch_vec_t<6>(job[0], job[1], st);
        case 7: return launch_vec_t<7>(job[0], job[1], st);
        default: return launch_vec_t<8>(job[0], job[1], st);
    }
}

// ------------------------------------------------------------------ token-tiled bulk kernel

constexpr int kTile = 128;            // tokens per CTA
constexpr int kBulkThreads = 512;
constexpr int kActLd = kD + 4;        // padded row of the activation tile (floats)
constexpr size_t kBulkSmem = (size_t)(kD * kHid + kHid * kHid + kHid * kBits) * 2   // bf16 weights
                             + (size_t)2 * kTile * kActLd * 4;                    // two activation tiles

// One hidden layer for a 64-token tile: thread (oq, tg) owns the four outputs 4 oq .. 4 oq + 3 of the eight tokens
// 8 tg .. 8 tg + 7 (32 independent chains).  Per four terms a thread reads four 8-byte weight groups and eight
// 16-byte activation groups (a warp = the 32 output groups of one token group: the activations are broadcasts)
// for 128 fmas, which leaves the layer bound by the fp32 pipe, not by shared memory.
__device__ __forceinline__ void bulk_hidden_layer(const float *__restrict__ in, float *__restrict__ out,
                                                  const uint16_t *__restrict__ w, const float *bias, int oq, int tg) {
    float z[8][4];
    {
        float b4[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) b4[j] = bias ? bias[4 * oq + j] : 0.0f;
#pragma unroll
        for (int t = 0; t < 8; ++t)
#pragma unroll
            for (int j = 0; j < 4; ++j) z[t][j] = b4[j];
    }
    const float *hin = in + (size_t)tg * 8 * kActLd;
#pragma unroll 4
    for (int k = 0; k < 128; k += 4) {
        float wf[4][4];   // [term][output]
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint2 wv = *reinterpret_cast<const uint2 *>(w + (k + i) * kHid + 4 * oq);
            wf[i][0] = __uint_as_float(wv.x << 16);
            wf[i][1] = __uint_as_float(wv.x & 0xffff0000u);
            wf[i][2] = __uint_as_float(wv.y << 16);
            wf[i][3] = __uint_as_float(wv.y & 0xffff0000u);
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const float4 hv = *reinterpret_cast<const float4 *>(hin + t * kActLd + k);   // warp broadcast
#pragma unroll
            for (int j = 0; j < 4; ++j) {   // ascending term index within every chain
                z[t][j] = __fmaf_rn(hv.x, wf[0][j], z[t][j]);
                z[t][j] = __fmaf_rn(hv.y, wf[1][j], z[t][j]);
                z[t][j] = __fmaf_rn(hv.z, wf[2][j], z[t][j]);
                z[t][j] = __fmaf_rn(hv.w, wf[3][j], z[t][j]);
            }
        }
    }
    float *hout = out + (size_t)tg * 8 * kActLd + 4 * oq;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        float4 r;
        r.x = (z[t][0] > 0.0f) ? z[t][0] : 0.0f;
        r.y = (z[t][1] > 0.0f) ? z[t][1] : 0.0f;
        r.z = (z[t][2] > 0.0f) ? z[t][2] : 0.0f;
        r.w = (z[t][3] > 0.0f) ? z[t][3] : 0.0f;
        *reinterpret_cast<float4 *>(hout + t * kActLd) = r;
    }
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

    const int oq = tid & 31, tg = tid >> 5;   // a warp: the 32 groups of four outputs, for one group of eight tokens
    bulk_hidden_layer(actA, actB, sw1, map.b1 ? map.b1 + net * kHid : nullptr, oq, tg);
    __syncthreads();
    bulk_hidden_layer(actB, actA, sw2, map.b2 ? map.b2 + net * kHid : nullptr, oq, tg);
    __syncthreads();

    // last layer: thread (op, tq) owns outputs 2 op, 2 op + 1 of the four tokens 4 tq .. 4 tq + 3; a half-warp
    // holds the 16 output pairs of one token group, so two ballots per token collect its 32 sign bits
    {
        const int lane = tid & 31, op = tid & 15, tq = tid >> 4;
        float z[4][2];
        const float b0 = map.b3 ? map.b3[net * kBits + 2 * op] : 0.0f, b1 = map.b3 ? map.b3[net * kBits + 2 * op + 1] : 0.0f;
#pragma unroll
        for (int t = 0; t < 4; ++t) { z[t][0] = b0; z[t][1] = b1; }
        const float *hin = actA + (size_t)tq * 4 * kActLd;
#pragma unroll 4
        for (int k = 0; k < 128; k += 4) {
            float wf[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t wv = *reinterpret_cast<const uint32_t *>(sw3 + (k + i) * kBits + 2 * op);
                wf[i][0] = __uint_as_float(wv << 16);
                wf[i][1] = __uint_as_float(wv & 0xffff0000u);
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const float4 hv = *reinterpret_cast<const float4 *>(hin + t * kActLd + k);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    z[t][j] = __fmaf_rn(hv.x, wf[0][j], z[t][j]);
                    z[t][j] = __fmaf_rn(hv.y, wf[1][j], z[t][j]);
                    z[t][j] = __fmaf_rn(hv.z, wf[2][j], z[t][j]);
                    z[t][j] = __fmaf_rn(hv.w, wf[3][j], z[t][j]);
                }
            }
        }
        uint32_t *cb = codes + (long long)b * c_sb + (long long)h * c_sh + t0;
        auto spread16 = [](uint32_t v) {   // bit i -> bit 2 i
            v = (v | (v << 8)) & 0x00ff00ffu;
            v = (v | (v << 4)) & 0x0f0f0f0fu;
            v = (v | (v << 2)) & 0x33333333u;
            v = (v | (v << 1)) & 0x55555555u;
            return v;
        };
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint32_t even = __ballot_sync(0xffffffffu, z[t][0] > 0.0f), odd = __ballot_sync(0xffffffffu, z[t][1] > 0.0f);
            const int shift = lane & 16;   // this half-warp's 16 bits of either ballot
            const uint32_t code = spread16((even >> shift) & 0xffffu) | (spread16((odd >> shift) & 0xffffu) << 1);
            const int tok = tq * 4 + t;
            if (op == 0 && tok < nt) cb[tok] = code;
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

// ------------------------------------------------------------------ signatures of 64 to 512 bits
//
// Eq. 2 with a last layer of 128 x b (the widths of the bit-width study and of the SCORE-latency table): the token
// tile, the two hidden layers and the arithmetic of every output are those of encode_bulk_kernel; the last layer
// runs block by block over 32 outputs at a time (its 128 x 32 slice of W3 staged in shared memory), and block c
// becomes the 32-bit half c % 2 of word c / 2 of the packed signature (bit j = bit j % 64 of word j / 64).
namespace ha {

__global__ void __launch_bounds__(kBulkThreads) encode_bulk_wide_kernel(MapView map, int n_bits, int heads_per_kv, TensorView x,
                                                                       int T, uint32_t *codes32, long long c_sb,
                                                                       long long c_sh, const int32_t *slot) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint16_t *sw1 = reinterpret_cast<uint16_t *>(smem);
    uint16_t *sw2 = sw1 + kD * kHid;
    uint16_t *sw3 = sw2 + kHid * kHid;                     // one 128 x 32 block of the last layer at a time
    float *actA = reinterpret_cast<float *>(sw3 + kHid * kBits);
    float *actB = actA + kTile * kActLd;

    const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int net = h / heads_per_kv;
    const int tid = threadIdx.x;
    const int t0 = tile * kTile;
    const int nt = min(kTile, T - t0);
    const int n_words = n_bits / 64;
    {
        const uint4 *g1 = reinterpret_cast<const uint4 *>(map.w1 + (size_t)net * kD * kHid);
        const uint4 *g2 = reinterpret_cast<const uint4 *>(map.w2 + (size_t)net * kHid * kHid);
        uint4 *s1 = reinterpret_cast<uint4 *>(sw1), *s2 = reinterpret_cast<uint4 *>(sw2);
        for (int i = tid; i < kD * kHid / 8; i += kBulkThreads) s1[i] = __ldg(g1 + i);
        for (int i = tid; i < kHid * kHid / 8; i += kBulkThreads) s2[i] = __ldg(g2 + i);
    }
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
    const int oq = tid & 31, tg = tid >> 5;
    bulk_hidden_layer(actA, actB, sw1, map.b1 ? map.b1 + net * kHid : nullptr, oq, tg);
    __syncthreads();
    bulk_hidden_layer(actB, actA, sw2, map.b2 ? map.b2 + net * kHid : nullptr, oq, tg);
    __syncthreads();

    const int lane = tid & 31, op = tid & 15, tq = tid >> 4;
    const uint16_t *g3 = map.w3 + (size_t)net * kHid * n_bits;
    // the token slot a signature goes to: its position in the tile, or the append slot of its sequence (T == 1)
    long long tok_base = t0;
    bool write_ok = true;
    if (slot) { const int sl = slot[b]; write_ok = sl >= 0; tok_base = sl; }
    uint32_t *cb = codes32 + 2 * ((long long)b * c_sb + (long long)h * c_sh + tok_base * n_words);
    for (int blk = 0; blk < n_bits / 32; ++blk) {
        // W3[:, 32 blk .. 32 blk + 31]: 128 rows of 64 bytes, one 16-byte piece per thread
        {
            const int r = tid >> 2, pc = tid & 3;
            reinterpret_cast<uint4 *>(sw3)[tid] = __ldg(reinterpret_cast<const uint4 *>(g3 + (size_t)r * n_bits + 32 * blk) + pc);
        }
        __syncthreads();
        float z[4][2];
        const float b0 = map.b3 ? map.b3[net * n_bits + 32 * blk + 2 * op] : 0.0f;
        const float b1 = map.b3 ? map.b3[net * n_bits + 32 * blk + 2 * op + 1] : 0.0f;
#pragma unroll
        for (int t = 0; t < 4; ++t) { z[t][0] = b0; z[t][1] = b1; }
        const float *hin = actA + (size_t)tq * 4 * kActLd;
#pragma unroll 4
        for (int k = 0; k < 128; k += 4) {
            float wf[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t wv = *reinterpret_cast<const uint32_t *>(sw3 + (k + i) * kBits + 2 * op);
                wf[i][0] = __uint_as_float(wv << 16);
                wf[i][1] = __uint_as_float(wv & 0xffff0000u);
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const float4 hv = *reinterpret_cast<const float4 *>(hin + t * kActLd + k);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    z[t][j] = __fmaf_rn(hv.x, wf[0][j], z[t][j]);
                    z[t][j] = __fmaf_rn(hv.y, wf[1][j], z[t][j]);
                    z[t][j] = __fmaf_rn(hv.z, wf[2][j], z[t][j]);
                    z[t][j] = __fmaf_rn(hv.w, wf[3][j], z[t][j]);
                }
            }
        }
        auto spread16 = [](uint32_t v) {   // bit i -> bit 2 i
            v = (v | (v << 8)) & 0x00ff00ffu;
            v = (v | (v << 4)) & 0x0f0f0f0fu;
            v = (v | (v << 2)) & 0x33333333u;
            v = (v | (v << 1)) & 0x55555555u;
            return v;
        };
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint32_t even = __ballot_sync(0xffffffffu, z[t][0] > 0.0f), odd = __ballot_sync(0xffffffffu, z[t][1] > 0.0f);
            const int shift = lane & 16;
            const uint32_t code = spread16((even >> shift) & 0xffffu) | (spread16((odd >> shift) & 0xffffu) << 1);
            const int tok = tq * 4 + t;
            if (op == 0 && tok < nt && write_ok) cb[2 * ((long long)tok * n_words) + blk] = code;
        }
        __syncthreads();   // the block of W3 is overwritten by the next one
    }
}

cudaError_t launch_encode_wide(const MapView &map, int n_bits, int heads_per_kv, TensorView x, int B, int H, int T,
                               uint64_t *codes, long long c_sb, long long c_sh, const int32_t *slot, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(encode_bulk_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBulkSmem);
    if (e != cudaSuccess) return e;
    dim3 grid((T + kTile - 1) / kTile, H, B);
    encode_bulk_wide_kernel<<<grid, kBulkThreads, kBulkSmem, st>>>(map, n_bits, heads_per_kv, x, T, reinterpret_cast<uint32_t *>(codes),
                                                                  c_sb, c_sh, slot);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha
