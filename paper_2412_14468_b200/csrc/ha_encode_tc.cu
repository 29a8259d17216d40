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

#include <cstring>
#include <cuda.h>   // CUtensorMap (types only; the encoder is fetched through the runtime)

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


// ------------------------------------------------------------------ tcgen05 version
//
// The same chain of three GEMMs on the fifth-generation tensor cores.  A tile of 128 tokens is
// M = 128 rows = the 128 lanes of tensor memory; threads r and r + 128 of a group own row r.
//   layer 1  D[128 x 128] = X W1 + b1   A = token tile in shared memory (K-major core matrices),
//                                       B = W1 in shared memory (N-major core matrices), 8 x K16;
//                                       the bias is one more K16 step: A = a constant tile whose
//                                       rows are (1, 1, 0, ...), B = two rows holding b1 as a bf16
//                                       pair hi + lo
//   epilogue threads read their row of D (tcgen05.ld), apply ReLU, split into a bf16 pair hi + lo
//            (cvt.rn.bf16x2) and write both to tensor memory as the next A operand (tcgen05.st)
//   layer 2  D = A_hi W2 + A_lo W2 + b2  A from tensor memory, 16 x K16 + the bias step
//   layer 3  D[128 x 32] likewise; the epilogue packs the 32 sign bits of a row into its code.
// Activations never leave tensor memory and registers.
// Two groups of 256 threads (two per token row, each converting half of the columns) work on alternate tiles with their own token buffers, their own half of
// tensor memory (D 128 + A_hi 64 + A_lo 64 columns) and their own mbarrier, so that one group's
// tensor-core work runs under the other group's epilogue.  A CTA stays with one network: its
// weights are loaded once.  MMAs are issued by the first thread of a group and tracked with
// tcgen05.commit; every wait is bounded: on a timeout the group raises HA_DEV_TIMEOUT in the status
// word and stops, and the CTA frees its tensor memory and returns.

constexpr int kU_GroupThreads = 256;              // two threads per token row: each converts half of the columns
constexpr int kU_Threads = 2 * kU_GroupThreads;   // two groups
constexpr int kU_KG = kD / 8 + 2;                 // k-groups of 8 rows per weight matrix: 16 + 2 for the bias step
constexpr int kU_WBytes = kU_KG * 2048;           // 36864: W1 or W2 as k-groups x 16 n-blocks x (8 x 16 B)
constexpr int kU_W3Bytes = kU_KG * 512;           // 9216
constexpr int kU_OnesBytes = 4096;                // [128 rows x 16 k] tile of (1, 1, 0, ...) rows
constexpr int kU_XLboPad = 2048 + 16;             // bytes between the k-chunks of a token tile copied by the threads: 16 row-groups
                                                  // x 128 B, plus one 16-byte slot so that the 16 chunks of a row fall into different banks
constexpr int kU_XBytes = 16 * kU_XLboPad;        // 33024 (a tile copied by TMA uses 16 x 2048 of it)
constexpr int kU_Smem = 2 * kU_WBytes + kU_W3Bytes + kU_OnesBytes + 4 * kU_XBytes;   // 219136
constexpr uint32_t kU_TmemCols = 512;
constexpr uint32_t kU_SlotCols = 256, kU_ColD = 0, kU_ColAhi = 128, kU_ColAlo = 192;   // per group

// 64-bit shared-memory matrix descriptor, no swizzle: start address, leading and stride byte offsets
// in 16-byte units, descriptor version 1 (bits 46-47), layout type 0 (bits 61-63).
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46);
}
// 32-bit instruction descriptor of kind::f16: fp32 accumulate (bits 4-5 = 1), A and B bf16 (bits 7-9 and
// 10-12 = 1), A K-major (bit 15 = 0), B N-major (bit 16 = 1), N / 8 in bits 17-22, M / 16 in bits 24-28.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                   "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
                   "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                   "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
// 16 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
                 ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
                   "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void group_sync(int group) { asm volatile("bar.sync %0, 256;" ::"r"(group + 1) : "memory"); }

// try_wait parks the warp for a bounded time instead of spinning, so a waiting group leaves the issue
// slots to the group that is converting; the number of attempts is bounded as well.
__device__ __forceinline__ bool mbar_wait_parity_bounded(uint32_t bar, uint32_t parity) {
    for (int it = 0; it < (1 << 18); ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// ReLU + split of two fp32 values into packed bf16 pairs: hi = round(max(v, 0)), lo = round(max(v, 0) - hi);
// the remainder keeps its sign (hi may have been rounded up).  Low half = first value.
__device__ __forceinline__ void relu_split_pair(float v0, float v1, uint32_t &hi, uint32_t &lo) {
    v0 = fmaxf(v0, 0.0f);
    v1 = fmaxf(v1, 0.0f);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(v1), "f"(v0));
    const float r0 = v0 - __uint_as_float(hi << 16), r1 = v1 - __uint_as_float(hi & 0xffff0000u);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(r1), "f"(r0));
}

// A whole token tile through the tensor map of x seen as [B][H][16 k-chunks][T][8]: the box of 8 x 128 x 16
// elements lands chunk after chunk, each as 128 consecutive 16-byte rows, which is the core-matrix layout
// the MMA descriptor names (k-chunk stride 2048 bytes).  One instruction per tile.
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap *tmap, int t0, int h, int b, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"(tmap), "r"(0), "r"(t0), "r"(0), "r"(h), "r"(b), "r"(bar) : "memory");
}

// kTma: token tiles arrive through TMA (one thread per group issues one box copy and the tile's mbarrier
// counts the bytes); otherwise every thread copies 16-byte pieces with cp.async.
template <bool kTma>
__global__ void __launch_bounds__(kU_Threads, 1) encode_umma_kernel(const __grid_constant__ CUtensorMap tmap, MapView map,
                                                                   int heads_per_kv, TensorView x, int B, int H, int T,
                                                                   int ctas_per_net, uint32_t *__restrict__ codes,
                                                                   long long c_sb, long long c_sh,
                                                                   uint32_t *__restrict__ status) {
    constexpr int kU_XLbo = kTma ? 2048 : kU_XLboPad;
    extern __shared__ __align__(1024) unsigned char usm[];
    unsigned char *sW1 = usm, *sW2 = sW1 + kU_WBytes, *sW3 = sW2 + kU_WBytes, *sOnes = sW3 + kU_W3Bytes,
                  *sX = sOnes + kU_OnesBytes;
    __shared__ __align__(8) unsigned long long s_mbar[2];
    __shared__ __align__(8) unsigned long long s_xbar[2][2];   // [group][buffer]: arrival of a token tile (TMA)
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_fail[2];
    const int tid = threadIdx.x, warp = tid >> 5, group = tid >> 8, gt = tid & 255;
    const int row = gt & 127, half = gt >> 7;   // thread (row, half) converts columns 64 half .. 64 half + 63 of its row
    const int tiles_per_row = (T + kTcTile - 1) / kTcTile;
    const int net = blockIdx.x / ctas_per_net, part = blockIdx.x % ctas_per_net;
    // tiles of this network in the order (head of the network, sequence, tile); this CTA takes a contiguous share
    const long long n_net = (long long)heads_per_kv * B * tiles_per_row;
    const long long w_lo = n_net * part / ctas_per_net, w_hi = n_net * (part + 1) / ctas_per_net;
    if (w_lo >= w_hi) return;

    if (tid == 0) {
        mbar_init(smem_u32(&s_mbar[0]), 1);
        mbar_init(smem_u32(&s_mbar[1]), 1);
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&s_xbar[0][0]) + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_fail[0] = 0;
        s_fail[1] = 0;
    }
    if (warp == 0) {   // one warp allocates the tensor memory and passes the allocation right on
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"(kU_TmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // ---- weights (N-major core matrices: element (k, n) at (k/8) * LBO + (n/8) * 128 + (k%8) * 16 + (n%8) * 2),
    // the bias rows k = 128 (hi) and 129 (lo) behind them, and the constant tile of ones
    {
        const unsigned char *g1 = reinterpret_cast<const unsigned char *>(map.w1 + (size_t)net * kD * kHid);
        const unsigned char *g2 = reinterpret_cast<const unsigned char *>(map.w2 + (size_t)net * kHid * kHid);
        const unsigned char *g3 = reinterpret_cast<const unsigned char *>(map.w3 + (size_t)net * kHid * kBits);
        for (int e = tid; e < kD * 16; e += kU_Threads) {   // 16 chunks of 8 outputs per row k
            const int k = e >> 4, nb = e & 15;
            const uint32_t off = (k >> 3) * 2048 + nb * 128 + (k & 7) * 16;
            cp_async16(smem_u32(sW1) + off, g1 + (size_t)e * 16, 16u);
            cp_async16(smem_u32(sW2) + off, g2 + (size_t)e * 16, 16u);
        }
        for (int e = tid; e < kHid * 4; e += kU_Threads) {  // 4 chunks per row k
            const int k = e >> 2, nb = e & 3;
            cp_async16(smem_u32(sW3) + (k >> 3) * 512 + nb * 128 + (k & 7) * 16, g3 + (size_t)e * 16, 16u);
        }
        cp_async_commit();
        // k-groups 16 and 17: zero, then the bias pair in rows 0 and 1 of k-group 16
        for (int i = tid; i < 4096 / 16; i += kU_Threads) {
            reinterpret_cast<uint4 *>(sW1 + 16 * 2048)[i] = make_uint4(0u, 0u, 0u, 0u);
            reinterpret_cast<uint4 *>(sW2 + 16 * 2048)[i] = make_uint4(0u, 0u, 0u, 0u);
            reinterpret_cast<uint4 *>(sOnes)[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        for (int i = tid; i < 1024 / 16; i += kU_Threads) reinterpret_cast<uint4 *>(sW3 + 16 * 512)[i] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
        auto put_bias = [&](unsigned char *base, const float *bias, int n) {
            const float v = bias ? __ldg(bias + n) : 0.0f;
            const float h = bf16_round(v);
            const __nv_bfloat16 bh = __float2bfloat16_rn(h), bl = __float2bfloat16_rn(v - h);
            unsigned char *p = base + (n >> 3) * 128 + (n & 7) * 2;
            *reinterpret_cast<uint16_t *>(p) = *reinterpret_cast<const uint16_t *>(&bh);        // row k = 128
            *reinterpret_cast<uint16_t *>(p + 16) = *reinterpret_cast<const uint16_t *>(&bl);   // row k = 129
        };
        if (tid < kHid) {
            put_bias(sW1 + 16 * 2048, map.b1 ? map.b1 + net * kHid : nullptr, tid);
            put_bias(sW2 + 16 * 2048, map.b2 ? map.b2 + net * kHid : nullptr, tid);
            // ones tile, K-major: row r at (r/8) * 128 + (r%8) * 16 of k-chunk 0 holds (1, 1, 0, 0, 0, 0, 0, 0)
            *reinterpret_cast<uint32_t *>(sOnes + (tid >> 3) * 128 + (tid & 7) * 16) = 0x3f803f80u;
        }
        if (tid < kBits) put_bias(sW3 + 16 * 512, map.b3 ? map.b3 + net * kBits : nullptr, tid);
    }
    cp_async_wait<0>();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // ordinary writes -> visible to the tensor cores
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base + group * kU_SlotCols;                 // this group's half
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);   // this warp's 32 lanes (warps w and w + 4 share them)
    const uint32_t bar = smem_u32(&s_mbar[group]);
    unsigned char *gX = sX + group * 2 * kU_XBytes;

    auto decode = [&](long long w, int &h, int &b, int &t0) {
        const long long per_head = (long long)B * tiles_per_row;
        const int hh = (int)(w / per_head);
        const long long r = w - (long long)hh * per_head;
        h = net * heads_per_kv + hh;
        b = (int)(r / tiles_per_row);
        t0 = (int)(r - (long long)b * tiles_per_row) * kTcTile;
    };
    // token tile, K-major core matrices: element (row r, k) at (k/8) * kU_XLbo + (r/8) * 128 + (r%8) * 16 + (k%8) * 2.
    // TMA: one box copy per tile; rows past T are filled with zeros by the tensor map.
    // Threads: a half-warp copies one 256-byte row (whole lines on the global side, 16 different banks on the
    // shared side thanks to the padded chunk stride).
    auto load_x = [&](long long w, int buf) {
        int h, b, t0;
        decode(w, h, b, t0);
        const uint32_t dst = smem_u32(gX + buf * kU_XBytes);
        if (kTma) {
            if (gt == 0) {
                const uint32_t xb = smem_u32(&s_xbar[group][buf]);
                mbar_expect_tx(xb, kTcTile * kD * 2);
                tma_load_tile(dst, &tmap, t0, h, b, xb);
            }
        } else {
            const unsigned char *src = reinterpret_cast<const unsigned char *>(x.ptr + (long long)b * x.sb + (long long)h * x.sh);
#pragma unroll
            for (int i = 0; i < kTcTile * 16 / kU_GroupThreads; ++i) {
                const int e = gt + i * kU_GroupThreads, r = e >> 4, ch = e & 15;
                const bool ok = t0 + r < T;
                cp_async16(dst + ch * kU_XLbo + (r >> 3) * 128 + (r & 7) * 16,
                           src + (long long)(ok ? t0 + r : 0) * x.sn * 2 + ch * 16, ok ? 16u : 0u);
            }
        }
    };

    constexpr uint32_t kIdesc128 = umma_idesc(128, 128), kIdesc32 = umma_idesc(128, 32);
    const uint64_t ones_desc = umma_desc(smem_u32(sOnes), 2048, 128);
    uint32_t phase = 0;
    // wait for the MMAs committed last; group-uniform result
    auto wait_mma = [&]() -> bool {
        const bool ok = mbar_wait_parity_bounded(bar, phase);
        phase ^= 1u;
        if (!ok) s_fail[group] = 1;
        tc_fence_after();
        group_sync(group);
        return s_fail[group] == 0;
    };
    // this thread's half row of the 128-column accumulator -> ReLU, hi / lo -> the A operand columns
    auto epilogue_hidden = [&]() {
        uint32_t v[2][32];   // both pieces are requested at once: one tensor-memory round trip
#pragma unroll
        for (int q = 0; q < 2; ++q) tmem_ld32(lane_base + kU_ColD + (2 * half + q) * 32, v[q]);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            uint32_t hi[16], lo[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
                relu_split_pair(__uint_as_float(v[q][2 * i]), __uint_as_float(v[q][2 * i + 1]), hi[i], lo[i]);
            tmem_st16(lane_base + kU_ColAhi + (2 * half + q) * 16, hi);
            tmem_st16(lane_base + kU_ColAlo + (2 * half + q) * 16, lo);
        }
        tmem_wait_st();
        tc_fence_before();
        group_sync(group);
    };

    bool failed = false;
    long long w = w_lo + group;
    if (w < w_hi) load_x(w, 0);
    cp_async_commit();
    int buf = 0;
    uint32_t xphase[2] = {0u, 0u};
    for (; w < w_hi; w += 2, buf ^= 1) {
        int h, b, t0;
        decode(w, h, b, t0);
        if (w + 2 < w_hi) load_x(w + 2, buf ^ 1);
        if (kTma) {             // this tile has landed when its mbarrier has counted all its bytes
            if (!mbar_wait_parity_bounded(smem_u32(&s_xbar[group][buf]), xphase[buf])) s_fail[group] = 1;
            xphase[buf] ^= 1u;
            group_sync(group);
            if (s_fail[group]) { failed = true; break; }
        } else {
            cp_async_commit();      // group of the next tile (empty after the last one)
            cp_async_wait<1>();     // this tile has landed
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            group_sync(group);
        }

        // ---- layer 1: D = X W1 + b1 (operands from shared memory), one MMA per 16 values of k
        if (gt == 0) {
            tc_fence_after();
            const uint32_t xa = smem_u32(gX + buf * kU_XBytes), wa = smem_u32(sW1);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                umma_ss(tmem + kU_ColD, umma_desc(xa + ks * 2 * kU_XLbo, kU_XLbo, 128), umma_desc(wa + ks * 4096, 2048, 128),
                        kIdesc128, ks > 0 ? 1u : 0u);
            umma_ss(tmem + kU_ColD, ones_desc, umma_desc(wa + 8 * 4096, 2048, 128), kIdesc128, 1u);
            umma_commit(bar);
        }
        if (!wait_mma()) { failed = true; break; }
        epilogue_hidden();

        // ---- layer 2: D = A_hi W2 + A_lo W2 + b2, A from tensor memory (8 columns per 16 values of k)
        if (gt == 0) {
            tc_fence_after();
            const uint32_t wa = smem_u32(sW2);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                umma_ts(tmem + kU_ColD, tmem + kU_ColAhi + ks * 8, umma_desc(wa + ks * 4096, 2048, 128), kIdesc128, ks > 0 ? 1u : 0u);
                umma_ts(tmem + kU_ColD, tmem + kU_ColAlo + ks * 8, umma_desc(wa + ks * 4096, 2048, 128), kIdesc128, 1u);
            }
            umma_ss(tmem + kU_ColD, ones_desc, umma_desc(wa + 8 * 4096, 2048, 128), kIdesc128, 1u);
            umma_commit(bar);
        }
        if (!wait_mma()) { failed = true; break; }
        epilogue_hidden();

        // ---- layer 3: D[128 x 32]
        if (gt == 0) {
            tc_fence_after();
            const uint32_t wa = smem_u32(sW3);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                umma_ts(tmem + kU_ColD, tmem + kU_ColAhi + ks * 8, umma_desc(wa + ks * 1024, 512, 128), kIdesc32, ks > 0 ? 1u : 0u);
                umma_ts(tmem + kU_ColD, tmem + kU_ColAlo + ks * 8, umma_desc(wa + ks * 1024, 512, 128), kIdesc32, 1u);
            }
            umma_ss(tmem + kU_ColD, ones_desc, umma_desc(wa + 8 * 1024, 512, 128), kIdesc32, 1u);
            umma_commit(bar);
        }
        if (!wait_mma()) { failed = true; break; }
        if (half == 0) {   // warp-uniform
            uint32_t v[32];
            tmem_ld32(lane_base + kU_ColD, v);
            tmem_wait_ld();
            uint32_t code = 0u;
#pragma unroll
            for (int o = 0; o < 32; ++o) code |= (__uint_as_float(v[o]) > 0.0f ? 1u : 0u) << o;
            if (t0 + row < T) codes[(long long)b * c_sb + (long long)h * c_sh + t0 + row] = code;
        }
        tc_fence_before();
        group_sync(group);   // the group is done with this token buffer and with D before they are reused
    }
    if (failed) {
        // A group that gave up still has work in flight: the tile it prefetched into the other buffer and,
        // after a timed-out MMA wait, the committed MMAs.  Give both one more bounded wait, so that nothing
        // lands in shared or tensor memory that this CTA has already given back.
        if (kTma && w + 2 < w_hi) mbar_wait_parity_bounded(smem_u32(&s_xbar[group][buf ^ 1]), xphase[buf ^ 1]);
        mbar_wait_parity_bounded(bar, phase ^ 1u);   // returns at once when no MMA is outstanding
        if (gt == 0 && status) atomicOr(status, HA_DEV_TIMEOUT);
    }
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(s_tmem_base), "r"(kU_TmemCols) : "memory");
    }
}

// Tensor map of x [B][H][T][128] (bf16, strides in elements) seen as [B][H][16][T][8], with boxes of
// 8 x 128 x 16 elements; false if the driver entry point is missing or the strides do not fit a tensor map.
static bool make_x_tensor_map(CUtensorMap *tm, TensorView x, int B, int H, int T) {
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn fn = nullptr;
    static bool looked = false;
    if (!looked) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
        else
            cudaGetLastError();
        looked = true;
    }
    if (!fn) return false;
    const cuuint64_t dims[5] = {8u, (cuuint64_t)T, (cuuint64_t)(kD / 8), (cuuint64_t)H, (cuuint64_t)B};
    const cuuint64_t strides[4] = {(cuuint64_t)x.sn * 2, 16u, (cuuint64_t)x.sh * 2, (cuuint64_t)x.sb * 2};   // bytes
    const cuuint32_t box[5] = {8u, (cuuint32_t)kTcTile, (cuuint32_t)(kD / 8), 1u, 1u}, estr[5] = {1u, 1u, 1u, 1u, 1u};
    for (int i = 0; i < 4; ++i)
        if (strides[i] == 0 || (strides[i] & 15)) return false;
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<uint16_t *>(x.ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_encode_umma(const MapView &map, int heads_per_kv, TensorView x, int B, int H, int T, uint32_t *codes,
                               long long c_sb, long long c_sh, uint32_t *status, cudaStream_t st) {
    const int n_nets = H / heads_per_kv;
    const long long n_net = (long long)heads_per_kv * B * ((T + kTcTile - 1) / kTcTile);   // tiles per network
    if (n_net <= 0 || n_nets <= 0) return cudaSuccess;
    long long per = sm_count() / n_nets;                 // CTAs per network: a CTA never changes its weights
    if (per < 1) per = 1;
    if (per > (n_net + 1) / 2) per = (n_net + 1) / 2;    // at least two tiles (one per group) for a CTA to be worth it
    if (per < 1) per = 1;
    CUtensorMap tm;
    memset(&tm, 0, sizeof(tm));
    const bool tma = make_x_tensor_map(&tm, x, B, H, T);
    cudaError_t e = tma ? cudaFuncSetAttribute(encode_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kU_Smem)
                        : cudaFuncSetAttribute(encode_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kU_Smem);
    if (e != cudaSuccess) return e;
    if (tma)
        encode_umma_kernel<true><<<(int)(n_nets * per), kU_Threads, kU_Smem, st>>>(tm, map, heads_per_kv, x, B, H, T, (int)per,
                                                                                  codes, c_sb, c_sh, status);
    else
        encode_umma_kernel<false><<<(int)(n_nets * per), kU_Threads, kU_Smem, st>>>(tm, map, heads_per_kv, x, B, H, T, (int)per,
                                                                                   codes, c_sb, c_sh, status);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha
