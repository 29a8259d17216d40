// ENCODE of whole prompts on the tensor cores (the step before the decode path: building the
// signature cache of Section 4.1 "Implementation" for n tokens at once; the paper names these
// matrix multiplications as the latency bottleneck at short contexts, Section 5.2).
//
// F = 128 -> 128 -> 128 -> 32 (Eq. 2) for a tile of 128 tokens is a chain of three small GEMMs.
// A warp owns 16 tokens and keeps their activations in registers from layer to layer: the fp32
// accumulator fragment of mma.m16n8k16 has exactly the layout of the next layer's A fragment, so
// nothing but the input tile and the weights ever touches shared memory.  Inputs and weights are
// bf16 and therefore exact operands; the fp32 hidden activations are fed to the next layer as a
// bf16 pair hi + lo (hi = round(h), lo = round(h - hi): 16 significant bits), two mma per product.
//
// Numerics: the sums are formed by the tensor cores in their own order and from 16-bit
// activations, not by the fp32 fused-multiply-add chain that defines the decode-step signatures.
// A bit can therefore differ from the chain's wherever the last layer's output is within ~1e-5 of
// zero; everywhere else the signatures are identical (the parity tests bound this by the margin of
// the exact output).  The chain-exact kernels in ha_encode.cu remain the reference for the decode
// step and are what ha_encode uses.
#include "ha_attn_dev.cuh"
#include "ha_encode_dev.cuh"

namespace ha {

constexpr int kTcTile = 128;                       // tokens per tile
constexpr int kTcThreads = 256;                    // 8 warps x 16 tokens
constexpr int kTcRow = kD * 2 + 16;                // padded row of the token tile and of W1 / W2 (bytes)
constexpr int kTcRow3 = kBits * 2 + 16;            // padded row of W3 (bytes)
constexpr int kTcW12Bytes = kD * kTcRow;           // 34816
constexpr int kTcW3Bytes = kHid * kTcRow3;         // 10240
constexpr int kTcXBytes = kTcTile * kTcRow;        // 34816
constexpr int kTcSmem = 2 * kTcW12Bytes + kTcW3Bytes + 2 * kTcXBytes;   // 149504

// hi / lo bf16 pair of two fp32 values after ReLU, packed for an A fragment register
__device__ __forceinline__ void split_relu(float v0, float v1, uint32_t &hi, uint32_t &lo) {
    v0 = fmaxf(v0, 0.0f);
    v1 = fmaxf(v1, 0.0f);
    const float h0 = bf16_round(v0), h1 = bf16_round(v1);
    hi = pack_bf16(h0, h1);
    lo = pack_bf16(v0 - h0, v1 - h1);
}

__global__ void __launch_bounds__(kTcThreads, 1) encode_tc_kernel(MapView map, int heads_per_kv, TensorView x, int B,
                                                                 int H, int T, uint32_t *__restrict__ codes,
                                                                 long long c_sb, long long c_sh) {
    extern __shared__ __align__(128) unsigned char tsm[];
    unsigned char *sW1 = tsm, *sW2 = sW1 + kTcW12Bytes, *sW3 = sW2 + kTcW12Bytes, *sX = sW3 + kTcW3Bytes;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int tiles_per_row = (T + kTcTile - 1) / kTcTile;
    const long long n_work = (long long)H * B * tiles_per_row;   // order: head-major, so that a CTA keeps its weights
    // contiguous range of work items per CTA
    const long long w_lo = n_work * blockIdx.x / gridDim.x, w_hi = n_work * (blockIdx.x + 1) / gridDim.x;
    if (w_lo >= w_hi) return;

    auto decode = [&](long long w, int &h, int &b, int &t0) {
        const long long per_head = (long long)B * tiles_per_row;
        h = (int)(w / per_head);
        const long long r = w - (long long)h * per_head;
        b = (int)(r / tiles_per_row);
        t0 = (int)(r - (long long)b * tiles_per_row) * kTcTile;
    };
    auto load_x = [&](long long w, int buf) {   // 128 rows x 16 chunks of 16 bytes; rows past T are zero-filled
        int h, b, t0;
        decode(w, h, b, t0);
        const unsigned char *src = reinterpret_cast<const unsigned char *>(x.ptr + (long long)b * x.sb + (long long)h * x.sh);
        const uint32_t dst = smem_u32(sX + buf * kTcXBytes);
#pragma unroll
        for (int i = 0; i < kTcTile * 16 / kTcThreads; ++i) {
            const int e = tid + i * kTcThreads, row = e >> 4, ch = e & 15;
            const bool ok = t0 + row < T;
            cp_async16(dst + row * kTcRow + ch * 16, src + (long long)(ok ? t0 + row : 0) * x.sn * 2 + ch * 16, ok ? 16u : 0u);
        }
    };
    auto load_weights = [&](int net) {
        const unsigned char *g1 = reinterpret_cast<const unsigned char *>(map.w1 + (size_t)net * kD * kHid);
        const unsigned char *g2 = reinterpret_cast<const unsigned char *>(map.w2 + (size_t)net * kHid * kHid);
        const unsigned char *g3 = reinterpret_cast<const unsigned char *>(map.w3 + (size_t)net * kHid * kBits);
        for (int e = tid; e < kD * 16; e += kTcThreads) {
            cp_async16(smem_u32(sW1) + (e >> 4) * kTcRow + (e & 15) * 16, g1 + (size_t)e * 16, 16u);
            cp_async16(smem_u32(sW2) + (e >> 4) * kTcRow + (e & 15) * 16, g2 + (size_t)e * 16, 16u);
        }
        for (int e = tid; e < kHid * 4; e += kTcThreads)
            cp_async16(smem_u32(sW3) + (e >> 2) * kTcRow3 + (e & 3) * 16, g3 + (size_t)e * 16, 16u);
    };

    // ldmatrix lane offsets.  A (token tile, row-major): matrix j = lane/8 -> rows (j&1)*8 + lane%8, k block j/2.
    const uint32_t a_off = (uint32_t)((((lane >> 3) & 1) * 8 + (lane & 7)) * kTcRow + (lane >> 4) * 16);
    // B (weights [k][n], transposed on load): matrix j -> k rows (j&1)*8 + lane%8, n block j/2.
    const uint32_t b_off12 = (uint32_t)((((lane >> 3) & 1) * 8 + (lane & 7)) * kTcRow + (lane >> 4) * 16);
    const uint32_t b_off3 = (uint32_t)((((lane >> 3) & 1) * 8 + (lane & 7)) * kTcRow3 + (lane >> 4) * 16);

    int cur_net = -1;
    load_x(w_lo, 0);
    cp_async_commit();
    int buf = 0;
    for (long long w = w_lo; w < w_hi; ++w, buf ^= 1) {
        int h, b, t0;
        decode(w, h, b, t0);
        const int net = h / heads_per_kv;
        if (net != cur_net) {   // CTA-uniform; the previous tile's math is behind the barrier at the end of the loop
            load_weights(net);
            cur_net = net;
        }
        cp_async_commit();      // group of the weights (empty when they stay)
        if (w + 1 < w_hi) load_x(w + 1, buf ^ 1);
        cp_async_commit();      // group of the next tile (empty after the last one)
        cp_async_wait<1>();     // everything but the next tile has landed: this tile and the weights
        __syncthreads();

        const float *bias1 = map.b1 ? map.b1 + net * kHid : nullptr;
        const float *bias2 = map.b2 ? map.b2 + net * kHid : nullptr;
        const float *bias3 = map.b3 ? map.b3 + net * kBits : nullptr;
        const uint32_t xs = smem_u32(sX + buf * kTcXBytes) + warp * 16 * kTcRow + a_off;

        // ---- layer 1: acc1[nt] = bias + X W1, n tile nt covers outputs 8 nt .. 8 nt + 7
        float acc1[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            const float b0 = bias1 ? __ldg(bias1 + 8 * nt + 2 * c) : 0.0f, b1 = bias1 ? __ldg(bias1 + 8 * nt + 2 * c + 1) : 0.0f;
            acc1[nt][0] = b0; acc1[nt][1] = b1; acc1[nt][2] = b0; acc1[nt][3] = b1;
        }
#pragma unroll
        for (int kt = 0; kt < 8; ++kt) {
            uint32_t a[4];
            ldmatrix_x4(a, xs + kt * 32);
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                uint32_t bw[4];
                ldmatrix_x4_trans(bw, smem_u32(sW1) + kt * 16 * kTcRow + np * 32 + b_off12);
                mma_bf16_16816(acc1[2 * np], a[0], a[1], a[2], a[3], bw[0], bw[1]);
                mma_bf16_16816(acc1[2 * np + 1], a[0], a[1], a[2], a[3], bw[2], bw[3]);
            }
        }
        // ---- layer 2: A fragments straight from acc1 (ReLU, hi + lo)
        float acc2[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            const float b0 = bias2 ? __ldg(bias2 + 8 * nt + 2 * c) : 0.0f, b1 = bias2 ? __ldg(bias2 + 8 * nt + 2 * c + 1) : 0.0f;
            acc2[nt][0] = b0; acc2[nt][1] = b1; acc2[nt][2] = b0; acc2[nt][3] = b1;
        }
#pragma unroll
        for (int kt = 0; kt < 8; ++kt) {
            uint32_t ah[4], al[4];
            split_relu(acc1[2 * kt][0], acc1[2 * kt][1], ah[0], al[0]);
            split_relu(acc1[2 * kt][2], acc1[2 * kt][3], ah[1], al[1]);
            split_relu(acc1[2 * kt + 1][0], acc1[2 * kt + 1][1], ah[2], al[2]);
            split_relu(acc1[2 * kt + 1][2], acc1[2 * kt + 1][3], ah[3], al[3]);
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                uint32_t bw[4];
                ldmatrix_x4_trans(bw, smem_u32(sW2) + kt * 16 * kTcRow + np * 32 + b_off12);
                mma_bf16_16816(acc2[2 * np], ah[0], ah[1], ah[2], ah[3], bw[0], bw[1]);
                mma_bf16_16816(acc2[2 * np], al[0], al[1], al[2], al[3], bw[0], bw[1]);
                mma_bf16_16816(acc2[2 * np + 1], ah[0], ah[1], ah[2], ah[3], bw[2], bw[3]);
                mma_bf16_16816(acc2[2 * np + 1], al[0], al[1], al[2], al[3], bw[2], bw[3]);
            }
        }
        // ---- layer 3: 32 outputs
        float acc3[4][4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float b0 = bias3 ? __ldg(bias3 + 8 * nt + 2 * c) : 0.0f, b1 = bias3 ? __ldg(bias3 + 8 * nt + 2 * c + 1) : 0.0f;
            acc3[nt][0] = b0; acc3[nt][1] = b1; acc3[nt][2] = b0; acc3[nt][3] = b1;
        }
#pragma unroll
        for (int kt = 0; kt < 8; ++kt) {
            uint32_t ah[4], al[4];
            split_relu(acc2[2 * kt][0], acc2[2 * kt][1], ah[0], al[0]);
            split_relu(acc2[2 * kt][2], acc2[2 * kt][3], ah[1], al[1]);
            split_relu(acc2[2 * kt + 1][0], acc2[2 * kt + 1][1], ah[2], al[2]);
            split_relu(acc2[2 * kt + 1][2], acc2[2 * kt + 1][3], ah[3], al[3]);
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                uint32_t bw[4];
                ldmatrix_x4_trans(bw, smem_u32(sW3) + kt * 16 * kTcRow3 + np * 32 + b_off3);
                mma_bf16_16816(acc3[2 * np], ah[0], ah[1], ah[2], ah[3], bw[0], bw[1]);
                mma_bf16_16816(acc3[2 * np], al[0], al[1], al[2], al[3], bw[0], bw[1]);
                mma_bf16_16816(acc3[2 * np + 1], ah[0], ah[1], ah[2], ah[3], bw[2], bw[3]);
                mma_bf16_16816(acc3[2 * np + 1], al[0], al[1], al[2], al[3], bw[2], bw[3]);
            }
        }
        // ---- sign bits: this lane holds outputs 8 nt + 2c, 8 nt + 2c + 1 of rows g and g + 8
        uint32_t m_lo = 0u, m_hi = 0u;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int bit = 8 * nt + 2 * c;
            m_lo |= (acc3[nt][0] > 0.0f ? 1u : 0u) << bit;
            m_lo |= (acc3[nt][1] > 0.0f ? 1u : 0u) << (bit + 1);
            m_hi |= (acc3[nt][2] > 0.0f ? 1u : 0u) << bit;
            m_hi |= (acc3[nt][3] > 0.0f ? 1u : 0u) << (bit + 1);
        }
        m_lo |= __shfl_xor_sync(0xffffffffu, m_lo, 1);
        m_lo |= __shfl_xor_sync(0xffffffffu, m_lo, 2);
        m_hi |= __shfl_xor_sync(0xffffffffu, m_hi, 1);
        m_hi |= __shfl_xor_sync(0xffffffffu, m_hi, 2);
        if (c == 0) {
            uint32_t *cb = codes + (long long)b * c_sb + (long long)h * c_sh + t0 + warp * 16;
            if (t0 + warp * 16 + g < T) cb[g] = m_lo;
            if (t0 + warp * 16 + g + 8 < T) cb[g + 8] = m_hi;
        }
        __syncthreads();   // every warp is done with this token buffer (and these weights) before they are overwritten
    }
}

cudaError_t launch_encode_tc(const MapView &map, int heads_per_kv, TensorView x, int B, int H, int T, uint32_t *codes,
                             long long c_sb, long long c_sh, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(encode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);
    if (e != cudaSuccess) return e;
    const long long n_work = (long long)H * B * ((T + kTcTile - 1) / kTcTile);
    if (n_work <= 0) return cudaSuccess;
    const int grid = (int)((n_work < sm_count()) ? n_work : sm_count());
    encode_tc_kernel<<<grid, kTcThreads, kTcSmem, st>>>(map, heads_per_kv, x, B, H, T, codes, c_sb, c_sh);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha
