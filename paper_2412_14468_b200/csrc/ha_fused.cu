// The whole layer-step in ONE launch, for small batches (as many (sequence, KV head) units as clusters
// are resident at once: on a 148-SM device 33 clusters of 8 CTAs or 71 of 4 with index lists of up to 1024
// entries, 15 clusters of 8 with longer lists) and sequences of up to 32768 tokens: ENCODE -> SCORE -> TOPK
// -> GATHER-ATT (Section 4 recipe, Section 4.1 "Implementation") with one thread-block cluster of CS
// CTAs per unit, so that a small-batch decode step has no kernel boundary or global-memory hand-off on
// its critical path:
//
//   P0  every CTA requests its slice of the signature cache; the encoding CTAs of the cluster fetch the
//       query-side / key-side mapping weights and store them transposed in shared memory; all of it
//       before the programmatic-launch wait, i.e. behind the preceding kernel.
//   P1  the first CTAs of the cluster encode the G query vectors (one per CTA when the cluster has room,
//       else 2 or 4), the next CTA the appended key (fp32 fma chains, Eq. 2, one chain per thread); the
//       signatures are stored into every CTA's shared memory (DSMEM); cluster barrier.
//   P2  scores as bytes in registers, per-CTA histogram stored into every CTA's table, cluster barrier,
//       threshold (every warp for itself), compaction of the CTA's slice; the parts of the index list
//       are stored into the shared memory of the CTAs that will attend to them (one-stage variant) or
//       into global memory; cluster barrier.
//   P3  each CTA takes a 1/CS of the list: rows fetched with 16-byte cp.async into per-warp
//       shared-memory stages, QK^T and PV on the tensor cores, online softmax; the CTA states
//       are written into CTA 0's shared memory (DSMEM stores), cluster barrier, CTA 0 merges,
//       normalises and rounds once to bf16.
// Every cross-CTA hand-off is a push followed by a hardware cluster barrier (no flag, no spin, no remote
// read).  Results are bit-identical to the multi-kernel path for signatures, counts and index lists;
// attention outputs agree within the usual fp32 reordering.
#include "ha_attn_dev.cuh"
#include "ha_encode_dev.cuh"
#include "ha_score_dev.cuh"

namespace ha {

constexpr int kFusedMaxCS = 8;                               // CTAs per cluster (template parameter CS: 8 or 4; 2 is supported, unused)
constexpr int kFusedWarps = 8;
constexpr int kFusedThreads = kFusedWarps * 32;
constexpr int kFusedMaxSeq = 32768;                          // 32 uint4 of signatures per thread position, shared by the cluster
constexpr int kFusedMaxStages = 2;                           // row blocks in flight per warp (template parameter S)
constexpr int kFusedWeightBytes = (kD * kHid + kHid * kHid + kHid * kBits) * 2;
constexpr int kFusedOneStageMaxK = 2048;                     // one-stage variant: longest index list
constexpr int kFusedListOffset = kFusedWarps * kStageBytes;  // one-stage variant: this CTA's part of the list sits behind the ring
// query vectors per encoding CTA: the smallest divisor of G that leaves the cluster one CTA for the appended key
__host__ __device__ constexpr int fused_q_per_cta(int G, int CS) {
    return (G <= CS - 1) ? 1 : (G / 2 <= CS - 1) ? 2 : (G / 4 <= CS - 1) ? 4 : 8;
}
// Dynamic shared memory of a CTA: [weights | S row stages per warp] union, activations, the CS CTA states
// of the G heads (used in CTA 0).  With S = 1 two CTAs fit one SM (and the kernel is compiled for 128
// registers): two consecutive steps are then resident together, each cluster of the later one already
// parked at its launch wait, whereas only 15 clusters of eight one-CTA SMs exist on the device.
__host__ __device__ constexpr int fused_ring_bytes(int S) { return kFusedWarps * S * kStageBytes; }
__host__ __device__ constexpr int fused_union_bytes(int S) { return fused_ring_bytes(S) > kFusedWeightBytes ? fused_ring_bytes(S) : kFusedWeightBytes; }
__host__ __device__ constexpr int fused_act_bytes(int G, int CS) { return 2 * fused_q_per_cta(G, CS) * kD * 4; }   // two activation buffers
__host__ __device__ constexpr int fused_part_bytes(int G, int CS) { return CS * G * (kD + 2) * 4; }
__host__ __device__ constexpr int fused_smem_bytes(int G, int S, int CS) {
    return fused_union_bytes(S) + fused_act_bytes(G, CS) + fused_part_bytes(G, CS);
}
static_assert(kFusedListOffset + kFusedOneStageMaxK / 2 * 4 <= kFusedWeightBytes, "the list part fits behind the one-stage ring");

struct FusedArgs {
    MapView map_q, map_k;
    const uint16_t *q, *k_new;
    TensorView K, V;
    uint32_t *k_codes;
    long long kc_sb, kc_sh;
    const int32_t *seq_lens, *k_per_seq;
    int k_uniform, max_seq_len, k_max, Hq, Hkv;
    Windows win;
    float scale_log2;
    uint32_t *q_codes;
    int32_t *idx;
    long long idx_sb, idx_sh;
    int32_t *count;
    uint16_t *out;
    float *lse;
    // paged K/V (block_table != NULL): token t of sequence b lives in page block_table[b*bt_sb + (t >> page_shift)],
    // slot t & (2^page_shift - 1); K.sb / V.sb are then the page strides and page_rows = K.sb / K.sn
    const int32_t *block_table;
    long long bt_sb;
    int page_shift, page_rows;
    // host-buffer entry: q, k_new and v_new are mapped host memory.  The kernel then appends the new K and V
    // rows itself (slot n - 1) and keeps a copy of the unit's queries in shared memory, so that each of them
    // crosses the bus once per CTA and never on the critical path of the attention phase.
    const uint16_t *v_new;
    uint32_t *status;   // stand-alone cluster gather: device status word (HA_DEV_BAD_INDEX)
};

__device__ __forceinline__ void st_dsmem_u32(uint32_t *local, uint32_t rank, uint32_t v) {
    uint32_t a = (uint32_t)__cvta_generic_to_shared(local), ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(ra), "r"(v) : "memory");
}
__device__ __forceinline__ void st_dsmem_f32(float *local, uint32_t rank, float v) {
    uint32_t a = (uint32_t)__cvta_generic_to_shared(local), ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}

// ENCODE of NV vectors that share one network by the first 128 threads of the CTA: thread o runs the
// chains of output o for every vector.  A second warp per scheduler would not shorten any chain.  The
// caller has put the three matrices into shared memory, transposed (TransposedFetch), before the
// call; the barrier that publishes the input vectors also publishes them.  Signature v is written to
// word v of `dst` in the shared memory of EVERY CTA of the cluster (lanes 0..CS-1 of the warp that holds it
// store to CTAs 0..CS-1; the cluster barrier that follows makes the stores visible).
template <int NV, int CS>
__device__ __forceinline__ void fused_encode(const uint16_t *x0, long long x_stride, const uint16_t *sw1,
                                             const uint16_t *sw2, const uint16_t *sw3, float *actA, float *actB,
                                             uint32_t *dst, float bias1, float bias2, float bias3) {
    const int tid = threadIdx.x, o = tid & 127;
    const bool active = tid < 128;
    if (active) {
#pragma unroll
        for (int v = 0; v < NV; ++v) actA[v * kD + o] = bf16_bits_to_float(__ldg(x0 + (long long)v * x_stride + o));
    }
    __syncthreads();
    float z[NV];
    if (active) {
#pragma unroll
        for (int v = 0; v < NV; ++v) z[v] = bias1;
        vec_layer_t<NV>(actA, sw1, o, z);
#pragma unroll
        for (int v = 0; v < NV; ++v) actB[v * kD + o] = (z[v] > 0.0f) ? z[v] : 0.0f;
    }
    __syncthreads();
    if (active) {
#pragma unroll
        for (int v = 0; v < NV; ++v) z[v] = bias2;
        vec_layer_t<NV>(actB, sw2, o, z);
#pragma unroll
        for (int v = 0; v < NV; ++v) actA[v * kD + o] = (z[v] > 0.0f) ? z[v] : 0.0f;
    }
    __syncthreads();
    {
        const int v = tid >> 5, lane = tid & 31;   // warp v encodes vector v, one output bit per lane
        if (v < NV) {
            float z3[1] = {bias3};
            vec_layer_t<1>(actA + v * kD, sw3, lane, z3);
            const uint32_t code = __ballot_sync(0xffffffffu, z3[0] > 0.0f);
            if (lane < CS) st_dsmem_u32(dst + v, (uint32_t)lane, code);
        }
    }
}

// GATHER-ATT over this CTA's share of a unit's index list, blocks [blk_lo, blk_hi) of 16 entries, and the merge
// of the cluster's CTA states in CTA 0, which writes the unit's outputs.  Shared by the fused step and the
// stand-alone cluster gather.  kLocalList: the CTA's part of the list sits in its shared memory (s_list), else
// in global memory (list).  kQShared: q_src is a copy of the unit's queries in shared memory.  kCheck: entries
// >= n_rows are skipped and reported through `bad` (lists that the caller wrote).
template <int G, int S, int CS, bool kLocalList, bool kQShared, bool kCheck>
__device__ __forceinline__ void fused_attention(const FusedArgs &a, uint32_t rank, int b, int kvh, long long head0, int keep,
                                                int n_rows, int blk_lo, int blk_hi, const int32_t *list,
                                                const int32_t *s_list, const uint16_t *q_src, unsigned char *ring,
                                                float *part_ml, float *part_acc, float (*s_m)[8], float (*s_l)[8],
                                                uint32_t (*s_mask)[kFusedMaxStages], bool &bad) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool paged = a.block_table != nullptr;   // rows are then addressed from the pool's base
    const unsigned char *Kb = reinterpret_cast<const unsigned char *>(a.K.ptr + (paged ? 0LL : (long long)b * a.K.sb) + (long long)kvh * a.K.sh);
    const unsigned char *Vb = reinterpret_cast<const unsigned char *>(a.V.ptr + (paged ? 0LL : (long long)b * a.V.sb) + (long long)kvh * a.V.sh);
    const int32_t *pages = paged ? a.block_table + (long long)b * a.bt_sb : nullptr;
    const long long k_row = a.K.sn * 2, v_row = a.V.sn * 2;
    unsigned char *my_ring = ring + warp * (S * kStageBytes);
    const uint32_t ring_u32 = smem_u32(my_ring);
    const int g = lane >> 2, cc = lane & 3;

    uint32_t qa[8][2];
    attn_load_q<G, kQShared>(qa, q_src, lane);
    float acc[8][4];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
    float m_run = -CUDART_INF_F, l_run = 0.0f;
    {
        // this warp's blocks: blk_lo + warp, + 8, ...; list entries were selected by peer CTAs: they sit in this
        // CTA's shared memory (one-stage variant) or are read from L2
        const int nblk = (blk_lo + warp < blk_hi) ? (blk_hi - blk_lo - warp + kFusedWarps - 1) / kFusedWarps : 0;
        auto token_of_block = [&](int i) -> int {
            const int p = (blk_lo + warp + i * kFusedWarps) * kBlockTokens + (lane & 15);
            int t = -1;
            if (i < nblk && p < keep) t = kLocalList ? s_list[p - blk_lo * kBlockTokens] : __ldcg(list + p);
            if (kCheck && t >= n_rows) { bad = true; t = -1; }   // a caller's list may point outside the sequence
            // paged: logical token -> row of the pool (page * rows per page stride + slot)
            if (paged && t >= 0) t = __ldg(pages + (t >> a.page_shift)) * a.page_rows + (t & ((1 << a.page_shift) - 1));
            return t;
        };
        auto issue = [&](int i, int stg) {
            const uint32_t valid = attn_issue_block(ring_u32 + stg * kStageBytes, Kb, Vb, k_row, v_row, token_of_block(i), lane);
            if (lane == 0) s_mask[warp][stg] = valid;
        };
        if (nblk > 0) issue(0, 0);
        cp_async_commit();
        for (int i = 0; i < nblk; ++i) {
            const int stg = (S > 1) ? (i & 1) : 0;
            if (S > 1) {   // the next block travels while this one is consumed
                if (i + 1 < nblk) issue(i + 1, stg ^ 1);
                cp_async_commit();
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            __syncwarp();
            const uint32_t ks = ring_u32 + stg * kStageBytes;
            attn_consume_block(ks, ks + kTileBytes, s_mask[warp][stg], qa, a.scale_log2, lane, acc, m_run, l_run);
            __syncwarp();
            if (S == 1) {   // one stage: the next block is requested once this one has been read
                if (i + 1 < nblk) issue(i + 1, 0);
                cp_async_commit();
            }
        }
        cp_async_wait<0>();
    }
    // merge the warps of this CTA through shared memory (each warp reuses its own ring)
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (cc == 0) { s_m[warp][g] = m_run; s_l[warp][g] = l_run; }
    __syncwarp();
    {
        float *my_acc = reinterpret_cast<float *>(my_ring);   // [G][128]
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int h = 2 * cc + hh;
            if (h < G) {
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    my_acc[h * kD + 16 * mt + g] = acc[mt][hh];
                    my_acc[h * kD + 16 * mt + 8 + g] = acc[mt][2 + hh];
                }
            }
        }
    }
    __syncthreads();
    {   // this CTA's state goes into slot `rank` of CTA 0's shared memory; the two thread halves share the heads
        const int d = tid & (kD - 1), hsel = tid >> 7;
#pragma unroll
        for (int j = 0; j < G; ++j) {
            if (G > 1 && (j & 1) != hsel) continue;
            if (G == 1 && hsel != 0) continue;
            float M = s_m[0][j];
#pragma unroll
            for (int w = 1; w < kFusedWarps; ++w) M = fmaxf(M, s_m[w][j]);
            float L = 0.0f, A = 0.0f;
            if (M > -CUDART_INF_F) {
#pragma unroll
                for (int w = 0; w < kFusedWarps; ++w) {
                    const float f = exp2f(s_m[w][j] - M);
                    L = fmaf(s_l[w][j], f, L);
                    A = fmaf(reinterpret_cast<const float *>(ring + w * (S * kStageBytes))[j * kD + d], f, A);
                }
            }
            st_dsmem_f32(part_acc + ((int)rank * G + j) * kD + d, 0, A);
            if (d == 0) {
                st_dsmem_f32(part_ml + ((int)rank * G + j) * 2, 0, M);
                st_dsmem_f32(part_ml + ((int)rank * G + j) * 2 + 1, 0, L);
            }
        }
    }
    cluster_sync_all();   // #4: the states of all CTAs have landed in CTA 0
    if (rank == 0) {
        const int d = tid & (kD - 1), hsel = tid >> 7;
#pragma unroll
        for (int j = 0; j < G; ++j) {
            if (G > 1 && (j & 1) != hsel) continue;
            if (G == 1 && hsel != 0) continue;
            float M = -CUDART_INF_F;
#pragma unroll
            for (int r = 0; r < CS; ++r) M = fmaxf(M, part_ml[(r * G + j) * 2]);
            float L = 0.0f, A = 0.0f;
            if (M > -CUDART_INF_F) {
#pragma unroll
                for (int r = 0; r < CS; ++r) {
                    const float f = exp2f(part_ml[(r * G + j) * 2] - M);
                    L = fmaf(part_ml[(r * G + j) * 2 + 1], f, L);
                    A = fmaf(part_acc[(r * G + j) * kD + d], f, A);
                }
            }
            const float o = (L > 0.0f) ? A / L : 0.0f;
            const __nv_bfloat16 ob = __float2bfloat16_rn(o);
            a.out[(head0 + j) * kD + d] = *reinterpret_cast<const uint16_t *>(&ob);
            if (a.lse && d == 0) a.lse[head0 + j] = (L > 0.0f) ? (M * kLn2 + logf(L)) : -CUDART_INF_F;
        }
    }
}

template <int G, int S, int CS, bool kHost>
__global__ void __launch_bounds__(kFusedThreads, S == 1 ? 2 : 1) fused_step_kernel(const FusedArgs a) {
    constexpr int kFusedUnionBytes = fused_union_bytes(S);
    constexpr int kFusedActBytes = fused_act_bytes(G, CS);
    constexpr int kL = kFusedMaxSeq / (CS * 4096) * 4;   // uint4 of signatures per thread: 4, 8 or 16
    constexpr int kFlagWords = (kL + 7) / 8;             // 32 tokens' flags per word
    constexpr int kQPer = fused_q_per_cta(G, CS);
    constexpr int kQCtas = G / kQPer;
    static_assert(kQCtas * kQPer == G && kQCtas < CS, "the cluster needs one more CTA for the appended key");
    constexpr bool kPreload = (CS > 2);   // signatures requested before the launch wait (16 uint4 would not fit the registers)
    extern __shared__ __align__(128) unsigned char fsm[];
    // dynamic: [weights | row ring] union, activations, the cluster's states (used in CTA 0)
    uint16_t *sw1 = reinterpret_cast<uint16_t *>(fsm);
    uint16_t *sw2 = sw1 + kD * kHid;
    uint16_t *sw3 = sw2 + kHid * kHid;
    unsigned char *ring = fsm;
    float *actA = reinterpret_cast<float *>(fsm + kFusedUnionBytes);
    float *actB = actA + kQPer * kD;
    float *part_ml = reinterpret_cast<float *>(fsm + kFusedUnionBytes + kFusedActBytes);   // [CS][G][2]
    float *part_acc = part_ml + CS * G * 2;                                   // [CS][G][128]
    __shared__ uint32_t s_codes[kMaxGroup + 1];   // the G query signatures and the appended key's, pushed by the encoding CTAs
    __shared__ uint32_t s_hist[kBins + 3];   // this CTA's histogram
    __shared__ int s_all[kFusedMaxCS][kBins + 3];   // the histograms of the cluster's CTAs, each pushed by its owner
    __shared__ __align__(16) uint32_t c_hist[kBins][32];   // one counter per (level, lane), shared by the warps
    __shared__ int s_wcnt[kFusedWarps];
    __shared__ float s_m[kFusedWarps][8], s_l[kFusedWarps][8];
    __shared__ uint32_t s_mask[kFusedWarps][kFusedMaxStages];

    cluster_arrive();   // completed below, before the first store into a peer's shared memory: every CTA has started
    const uint32_t rank = cluster_rank();
    const int kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Hq = a.Hq, Hkv = a.Hkv;
    const int n = max(min(a.seq_lens[b], a.max_seq_len), 0);
    int k = a.k_per_seq ? a.k_per_seq[b] : a.k_uniform;
    const WindowBounds wbd = window_bounds(a.win, n);   // always-kept tokens: byte kForcedByte, not counted
    const int n_forced = forced_before(wbd, n);
    const int keep_rest = max(0, min(min(k, a.k_max - n_forced), n - n_forced));   // heavy tokens among the others
    const int keep = n_forced + keep_rest;
    const long long head0 = (long long)b * Hq + (long long)kvh * G;
    uint32_t *row = a.k_codes + (long long)b * a.kc_sb + (long long)kvh * a.kc_sh;
    const bool has_new_key = (a.k_new != nullptr) && n > 0;

    // ---------------- P0: requests that do not depend on earlier kernels
    const int Lb = (n + CS * 1024 - 1) / (CS * 1024);
    const int wbase = ((int)rank * 1024 + warp * 128 + lane * 4) * Lb;
    uint4 c[kL];
    auto load_signatures = [&]() {
#pragma unroll
        for (int p = 0; p < kL; ++p) {
            const int base = wbase + p * 4;
            c[p] = (p < Lb && base < n) ? load_codes4(row, base, n) : make_uint4(0, 0, 0, 0);
        }
    };
    if (kPreload) load_signatures();
    // ENCODE roles: CTA r < kQCtas encodes kQPer query vectors (one per CTA while the cluster has room),
    // CTA kQCtas encodes the appended key; the other CTAs only scan
    const bool enc_q = (int)rank < kQCtas, enc_k = ((int)rank == kQCtas) && has_new_key;
    const bool encodes = enc_q || enc_k;
    const MapView &map = enc_q ? a.map_q : a.map_k;
    if (encodes) {   // the mapping's matrices do not depend on earlier kernels: fetched, transposed, behind them
        TransposedFetch<kFusedThreads, kHid> f1, f2;
        TransposedFetch<kFusedThreads, kBits> f3;
        f1.load(map.w1 + (size_t)kvh * kD * kHid, tid);   // all loads in flight before the first store
        f2.load(map.w2 + (size_t)kvh * kHid * kHid, tid);
        f3.load(map.w3 + (size_t)kvh * kHid * kBits, tid);
        f1.store(sw1, tid);
        f2.store(sw2, tid);
        f3.store(sw3, tid);
    }
    // biases are weights: they are fetched before the wait, like the matrices.  The vector to encode may
    // still be written by the kernel in front of this one, so it is only pulled into L2 here (a hint: the
    // writer's store updates the same L2 line) and read after the wait.
    float bias1 = 0.0f, bias2 = 0.0f, bias3 = 0.0f;
    if (encodes) {
        const int o = tid & 127;
        if (map.b1) bias1 = __ldg(map.b1 + kvh * kHid + o);
        if (map.b2) bias2 = __ldg(map.b2 + kvh * kHid + o);
        if (map.b3) bias3 = __ldg(map.b3 + kvh * kBits + (tid & (kBits - 1)));
        if (!kHost && tid < 2 * (enc_q ? kQPer : 1)) {   // 256 bytes per vector
            const uint16_t *xv = enc_q ? a.q + (head0 + kQPer * (int)rank) * kD : a.k_new + ((long long)b * Hkv + kvh) * kD;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(xv) + 128 * tid));
        }
    }
    for (int i = tid; i < kBins * 32 / 4; i += kFusedThreads)
        reinterpret_cast<uint4 *>(&c_hist[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    pdl_wait();                  // q, k_new and everything older in the stream is final from here on
    pdl_launch_dependents();
    cluster_wait();              // #0: all CTAs of the cluster are running (their shared memory may be written)
    uint4 q_stage = make_uint4(0u, 0u, 0u, 0u);
    if (kHost) {
        // the unit's G query vectors (16 bytes per thread) start their way across the bus now and are parked in
        // shared memory once the encoders are done with it
        if (tid < G * 16) q_stage = __ldg(reinterpret_cast<const uint4 *>(a.q + head0 * kD) + tid);
        if (enc_k && a.v_new && tid < 64) {   // the appended rows: 32 threads x 8 bytes for K, 32 for V (contiguous cache only)
            const int t = tid & 31;
            const long long src = ((long long)b * Hkv + kvh) * kD;
            const TensorView &X = (tid < 32) ? a.K : a.V;
            const uint2 v = __ldg(reinterpret_cast<const uint2 *>(((tid < 32) ? a.k_new : a.v_new) + src) + t);
            // slot seq_len - 1 as the stand-alone append kernel takes it (n is the length clamped to max_seq_len)
            uint16_t *dst = const_cast<uint16_t *>(X.ptr) + (long long)b * X.sb + (long long)kvh * X.sh + (long long)(a.seq_lens[b] - 1) * X.sn;
            reinterpret_cast<uint2 *>(dst)[t] = v;
        }
    }

    // ---------------- P1: ENCODE in the first kQCtas CTAs (queries) and the next one (appended key)
    if (enc_q) {
        fused_encode<kQPer, CS>(a.q + (head0 + kQPer * (int)rank) * kD, kD, sw1, sw2, sw3, actA, actB,
                            s_codes + kQPer * (int)rank, bias1, bias2, bias3);
    } else if (enc_k) {
        fused_encode<1, CS>(a.k_new + ((long long)b * Hkv + kvh) * kD, kD, sw1, sw2, sw3, actA, actB, s_codes + G, bias1,
                        bias2, bias3);
    }
    cluster_sync_all();   // #1: every CTA holds all signatures (and its counters are zeroed)
    // the signatures also go to global memory (outputs of the step; nobody in this kernel reads them there):
    // stored after the barrier, so that its release had nothing but shared-memory stores to wait for
    if (enc_q && tid < kQPer) a.q_codes[head0 + kQPer * (int)rank + tid] = s_codes[kQPer * (int)rank + tid];
    if (enc_k && tid == 0) row[n - 1] = s_codes[G];
    if (kHost && tid < G * 16) reinterpret_cast<uint4 *>(actA)[tid] = q_stage;   // the activations are dead
    uint32_t qc[G];
#pragma unroll
    for (int j = 0; j < G; ++j) qc[j] = s_codes[j];
    if (!kPreload) load_signatures();
    // Signatures that the early request may have seen in a stale state: slot n-1 (this step's appended token:
    // encoded above, or, when the step has no k_new, possibly written by an ha_encode call directly in front)
    // and slot n-2 (appended by a layer-step on the same cache directly in front, whose kernel lets this one
    // start before it has stored its signature).  Everything older was complete before this kernel started.
    auto replace_slot = [&](int t, uint32_t kc) {
#pragma unroll
        for (int p = 0; p < kL; ++p) {
            const int e = t - (wbase + p * 4);
            if (p < Lb && e >= 0 && e <= 3) {
                if (e == 0) c[p].x = kc; else if (e == 1) c[p].y = kc; else if (e == 2) c[p].z = kc; else c[p].w = kc;
            }
        }
    };
    if (has_new_key) replace_slot(n - 1, s_codes[G]);
    if (kPreload) {
        const int lo = wbase, hi = wbase + 4 * Lb;   // this lane's tokens (contiguous)
        if (!has_new_key && n - 1 >= lo && n - 1 < hi) replace_slot(n - 1, __ldcg(row + n - 1));
        if (n - 2 >= lo && n - 2 < hi) replace_slot(n - 2, __ldcg(row + n - 2));
    }

    // ---------------- P2: SCORE, histogram, threshold, compaction
    uint32_t sc[kL];
    {
        // a lane only meets its own column of counters, so an instruction never conflicts with itself; the
        // adds are reductions that never wait for a result.  The counter of score s sits (32 - s) rows
        // below the lane's counter of level 32: the address comes straight from the Hamming distance.
        const uint32_t top = (uint32_t)__cvta_generic_to_shared(&c_hist[kBins - 1][lane]);
        auto bump = [&](int ham) { asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(top - (uint32_t)ham * 128u) : "memory"); };
        auto hamming = [&](uint32_t code) {
            int h = __popc(code ^ qc[0]);
#pragma unroll
            for (int j = 1; j < G; ++j) h = min(h, __popc(code ^ qc[j]));
            return h;
        };
#pragma unroll
        for (int p = 0; p < kL; ++p) {
            const int base = wbase + p * 4;
            const int h0 = hamming(c[p].x), h1 = hamming(c[p].y), h2 = hamming(c[p].z), h3 = hamming(c[p].w);
            // bytes 33 - h = score + 1 (0 marks "no token"); no byte borrows because h <= 32
            uint32_t s4 = 0x21212121u - ((uint32_t)h0 | ((uint32_t)h1 << 8) | ((uint32_t)h2 << 16) | ((uint32_t)h3 << 24));
            if (p < Lb && base + 3 < n && base >= wbd.sink_end && base + 4 <= wbd.local_begin) {
                bump(h0); bump(h1); bump(h2); bump(h3);
            } else {
                const int hh[4] = {h0, h1, h2, h3};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int t = base + e;
                    if (p >= Lb || t >= n) s4 &= ~(0xffu << (8 * e));                      // zero byte: no token
                    else if (t < wbd.sink_end || t >= wbd.local_begin) s4 = (s4 & ~(0xffu << (8 * e))) | (kForcedByte << (8 * e));
                    else bump(hh[e]);
                }
            }
            sc[p] = s4;
        }
    }
    __syncthreads();
    // Fold and exchange: eight threads per level add four counters each and a shuffle tree completes the
    // level; then warp w stores the 33 counts into row `rank` of CTA w's table (one destination per warp, so
    // that a store instruction travels as one packet).
    for (int i = tid; i < kBins * 8; i += kFusedThreads) {   // 264 = 33 aligned groups of eight lanes
        const uint4 v = reinterpret_cast<const uint4 *>(&c_hist[i >> 3][0])[i & 7];
        uint32_t ssum = (v.x + v.y) + (v.z + v.w);
        const unsigned grp = 0xffu << (lane & 24);
        ssum += __shfl_xor_sync(grp, ssum, 1);
        ssum += __shfl_xor_sync(grp, ssum, 2);
        ssum += __shfl_xor_sync(grp, ssum, 4);
        if ((i & 7) == 0) s_hist[i >> 3] = ssum;
    }
    __syncthreads();
    if (warp < CS) {
        st_dsmem_u32(reinterpret_cast<uint32_t *>(&s_all[rank][lane]), (uint32_t)warp, s_hist[lane]);
        if (lane == 0) st_dsmem_u32(reinterpret_cast<uint32_t *>(&s_all[rank][32]), (uint32_t)warp, s_hist[32]);
    }
    cluster_sync_all();   // #2: every CTA holds all histograms of the cluster
    // every warp derives the threshold for itself (lane l owns level l, level 32 is read by every lane)
    int T, r, gt_before, eq_before;
    {
        int tot = 0, bef = 0, tot32 = 0, bef32 = 0;
#pragma unroll
        for (int rr = 0; rr < CS; ++rr) {
            const int v = s_all[rr][lane], v32 = s_all[rr][32];
            tot += v;
            tot32 += v32;
            if (rr < (int)rank) { bef += v; bef32 += v32; }
        }
        find_threshold(tot, bef, tot32, bef32, keep_rest, lane, T, r, gt_before, eq_before);
    }
    int32_t *list = a.idx + (long long)b * a.idx_sb + (long long)kvh * a.idx_sh;
    // GATHER-ATT shares: CTA c attends to blocks [c * bpc, (c + 1) * bpc) of the list (16 entries each)
    const int blocks_total = (keep + kBlockTokens - 1) / kBlockTokens;
    const int bpc = (blocks_total + CS - 1) / CS;                         // blocks per CTA
    const int blk_lo = min(blocks_total, (int)rank * bpc), blk_hi = min(blocks_total, blk_lo + bpc);
    // One-stage variant (at most kFusedOneStageMaxK entries): the selected tokens of this CTA's slice, which are a run of
    // consecutive list positions, are compacted in shared memory and sent, coalesced, into the shared memory
    // of the CTAs that will attend to them; each CTA writes its own part of the list to global memory after
    // the barrier.  Nothing but shared-memory stores is pending at the barrier and nobody reads the list from L2.
    constexpr bool kLocalList = (S == 1);
    int32_t *s_sel = reinterpret_cast<int32_t *>(fsm);                       // weights are dead, the ring not yet in use
    int32_t *s_list = reinterpret_cast<int32_t *>(fsm + kFusedListOffset);   // this CTA's part of the list, behind the ring
    if (!kLocalList && rank == 0) {
        if (tid == 0) a.count[b * Hkv + kvh] = keep;
        for (int i = keep + tid; i < a.k_max; i += kFusedThreads) list[i] = -1;
    }
    if (keep > 0) {
        // Per byte b = score + 1 (0 = no token): b + 127 - (T+1) sets bit 7 iff score > T, b + 128 - (T+1) iff
        // score >= T (no byte sum reaches 256).
        const uint32_t T4 = (uint32_t)(T + 1) * 0x01010101u;
        const uint32_t c_gt = 0x7f7f7f7fu - T4, c_ge = 0x80808080u - T4;
        uint32_t gtw[kFlagWords], eqw[kFlagWords];   // flags of this lane's 4 kL consecutive tokens, 32 per word
#pragma unroll
        for (int w = 0; w < kFlagWords; ++w) { gtw[w] = 0u; eqw[w] = 0u; }
#pragma unroll
        for (int p = 0; p < kL; ++p) {
            gtw[p / 8] |= high_bits_to_nibble(sc[p] + c_gt) << (4 * (p % 8));
            eqw[p / 8] |= high_bits_to_nibble(sc[p] + c_ge) << (4 * (p % 8));
        }
        int tot_packed = 0;
#pragma unroll
        for (int w = 0; w < kFlagWords; ++w) {
            eqw[w] ^= gtw[w];   // score > T implies score >= T
            tot_packed += __popc(gtw[w]) | (__popc(eqw[w]) << 16);
        }
        int winc = tot_packed;
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, winc, dd);
            if (lane >= dd) winc += v;
        }
        if (lane == 31) s_wcnt[warp] = winc;
        __syncthreads();
        // tokens before this warp's range with S > T (always-kept tokens count as such) / S == T
        const int cta_gt = gt_before + forced_before(wbd, min((int)rank * 1024 * Lb, n)), cta_eq = eq_before;
        int run_gt = cta_gt, run_eq = cta_eq, all_gt = cta_gt, all_eq = cta_eq;
#pragma unroll
        for (int w = 0; w < kFusedWarps; ++w) {
            const int wg = s_wcnt[w] & 0xffff, wq = (int)((unsigned)s_wcnt[w] >> 16);
            if (w < warp) { run_gt += wg; run_eq += wq; }
            all_gt += wg;
            all_eq += wq;
        }
        const int excl = winc - tot_packed;
        int g_run = run_gt + (excl & 0xffff), q_run = run_eq + (int)((unsigned)excl >> 16);
        if (kLocalList) {
            const int pos0 = cta_gt + min(cta_eq, r), cnt = all_gt + min(all_eq, r) - pos0;   // this CTA's run of positions
#pragma unroll
            for (int w = 0; w < kFlagWords; ++w)
                visit_selected32(wbase + 32 * w, gtw[w], eqw[w], g_run, q_run, r, [&](int pos, int t) { s_sel[pos - pos0] = t; });
            __syncthreads();
            const int per_cta = bpc * kBlockTokens;
            for (int i = tid; i < cnt; i += kFusedThreads) {
                const int pos = pos0 + i, owner = pos / per_cta;
                st_dsmem_u32(reinterpret_cast<uint32_t *>(&s_list[pos - owner * per_cta]), (uint32_t)owner, (uint32_t)s_sel[i]);
            }
        } else {
#pragma unroll
            for (int w = 0; w < kFlagWords; ++w) write_selected32(list, wbase + 32 * w, gtw[w], eqw[w], g_run, q_run, r);
        }
    }
    cluster_sync_all();   // #3: the index list is complete and visible to the whole cluster
    if (kLocalList) {
        const int my_lo = blk_lo * kBlockTokens, my_n = min(keep, blk_hi * kBlockTokens) - my_lo;
        for (int i = tid; i < my_n; i += kFusedThreads) list[my_lo + i] = s_list[i];
        if (rank == 0) {
            if (tid == 0) a.count[b * Hkv + kvh] = keep;
            for (int i = keep + tid; i < a.k_max; i += kFusedThreads) list[i] = -1;
        }
    }

    // ---------------- P3: GATHER-ATT over this CTA's share of the list, merge, output
    bool bad = false;
    fused_attention<G, S, CS, kLocalList, kHost, false>(a, rank, b, kvh, head0, keep, n, blk_lo, blk_hi, list, s_list,
                                                        kHost ? reinterpret_cast<const uint16_t *>(actA) : a.q + head0 * kD,
                                                        ring, part_ml, part_acc, s_m, s_l, s_mask, bad);
}

// ------------------------------------------------------------------ stand-alone GATHER-ATT with clusters
//
// ha_gather_attn for few units and short lists: the attention phase of the fused step on a list that the caller
// provides (one cluster of 8, 4 or 2 CTAs per (sequence, KV head), each CTA its share of the list, states merged in
// CTA 0's shared memory), instead of the persistent split-K kernel whose work split and global-memory merge cost
// more than the attention itself at this size.
__host__ __device__ constexpr int gather_cluster_smem_bytes(int G, int CS) { return fused_ring_bytes(1) + fused_part_bytes(G, CS); }

template <int G, int CS>
__global__ void __launch_bounds__(kFusedThreads, 2) gather_cluster_kernel(const FusedArgs a) {
    extern __shared__ __align__(128) unsigned char gsm[];
    unsigned char *ring = gsm;
    float *part_ml = reinterpret_cast<float *>(gsm + fused_ring_bytes(1));   // [CS][G][2]
    float *part_acc = part_ml + CS * G * 2;                                  // [CS][G][128]
    __shared__ float s_m[kFusedWarps][8], s_l[kFusedWarps][8];
    __shared__ uint32_t s_mask[kFusedWarps][kFusedMaxStages];
    cluster_arrive();   // completed before the first store into CTA 0's shared memory: every CTA has started
    const uint32_t rank = cluster_rank();
    const int kvh = blockIdx.y, b = blockIdx.z;
    const long long head0 = (long long)b * a.Hq + (long long)kvh * G;
    pdl_launch_dependents();
    pdl_wait();   // the list, its length and the rows may come from the kernels in front
    cluster_wait();
    const int n = a.seq_lens[b];
    const int keep = max(0, min(a.count[b * a.Hkv + kvh], a.k_max));
    const int blocks_total = (keep + kBlockTokens - 1) / kBlockTokens;
    const int bpc = (blocks_total + CS - 1) / CS;
    const int blk_lo = min(blocks_total, (int)rank * bpc), blk_hi = min(blocks_total, blk_lo + bpc);
    const int32_t *list = a.idx + (long long)b * a.idx_sb + (long long)kvh * a.idx_sh;
    bool bad = false;
    fused_attention<G, 1, CS, false, false, true>(a, rank, b, kvh, head0, keep, n, blk_lo, blk_hi, list, nullptr,
                                                  a.q + head0 * kD, ring, part_ml, part_acc, s_m, s_l, s_mask, bad);
    if (bad) atomicOr(a.status, HA_DEV_BAD_INDEX);
}

template <int G, int CS>
static void gather_cluster_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute (&attr)[2], int Hkv, int B, cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(CS, Hkv, B);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = gather_cluster_smem_bytes(G, CS);
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
}

// Opt in to the shared-memory carve-out (once per device); returns how many clusters the device holds at once.
template <int G, int CS>
static int gather_cluster_prepare() {
    static int clusters[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!clusters[dev]) {
        if (cudaFuncSetAttribute(gather_cluster_kernel<G, CS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 gather_cluster_smem_bytes(G, CS)) != cudaSuccess)
            return 0;
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[2];
        gather_cluster_config<G, CS>(cfg, attr, 1, 64, nullptr);
        cfg.numAttrs = 1;   // the cluster shape is all the occupancy query looks at
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gather_cluster_kernel<G, CS>, &cfg) != cudaSuccess || n <= 0) return 0;
        clusters[dev] = n;
    }
    return clusters[dev];
}

// Cluster size for `units` units: 8 while that many clusters are resident at once, else 4, else 2, else 0 (not
// eligible).  Unlike the fused step, whose clusters of 2 lose to the three-kernel path, the attention phase alone
// beats the split-K kernel at every cluster size (c3: 27.7 against 32.0 us with 128 clusters of 2).
template <int G>
static int gather_cluster_size(long long units) {
    if (units <= gather_cluster_prepare<G, 8>()) return 8;
    if (units <= gather_cluster_prepare<G, 4>()) return 4;
    if (units <= gather_cluster_prepare<G, 2>()) return 2;
    return 0;
}

// Lists of up to 2048 entries (a few blocks per warp) and as many units as clusters are resident at once.
bool gather_cluster_eligible(int B, int Hq, int Hkv, int k_max) {
    if (Hkv <= 0 || k_max > kFusedOneStageMaxK) return false;
    const long long units = (long long)B * Hkv;
    switch (Hq / Hkv) {
        case 1: return gather_cluster_size<1>(units) > 0;
        case 2: return gather_cluster_size<2>(units) > 0;
        case 4: return gather_cluster_size<4>(units) > 0;
        case 8: return gather_cluster_size<8>(units) > 0;
        default: return false;
    }
}

template <int G, int CS>
static cudaError_t launch_gather_cluster_gc(const FusedArgs &args, int B, cudaStream_t st) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    gather_cluster_config<G, CS>(cfg, attr, args.Hkv, B, st);
    cudaError_t e = cudaLaunchKernelEx(&cfg, gather_cluster_kernel<G, CS>, args);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

template <int G>
static cudaError_t launch_gather_cluster_g(const FusedArgs &args, int B, cudaStream_t st) {
    const int cs = gather_cluster_size<G>((long long)B * args.Hkv);
    if (cs == 8) return launch_gather_cluster_gc<G, 8>(args, B, st);
    if (cs == 4) return launch_gather_cluster_gc<G, 4>(args, B, st);
    if (cs == 2) return launch_gather_cluster_gc<G, 2>(args, B, st);
    return cudaErrorInvalidConfiguration;
}

cudaError_t launch_gather_cluster(int B, int Hq, int Hkv, float sm_scale, const uint16_t *q, TensorView K, TensorView V,
                                  const int32_t *seq_lens, const int32_t *idx, long long idx_sb, long long idx_sh,
                                  const int32_t *count, int k_max, uint16_t *out, float *lse, uint32_t *status,
                                  cudaStream_t st, const int32_t *block_table, long long bt_sb, int page_shift) {
    FusedArgs a{};
    a.block_table = block_table; a.bt_sb = bt_sb; a.page_shift = page_shift;
    a.page_rows = (block_table && K.sn > 0) ? (int)(K.sb / K.sn) : 0;
    a.q = q; a.K = K; a.V = V; a.seq_lens = seq_lens; a.k_max = k_max; a.Hq = Hq; a.Hkv = Hkv;
    a.scale_log2 = sm_scale * kLog2e; a.idx = const_cast<int32_t *>(idx); a.idx_sb = idx_sb; a.idx_sh = idx_sh;
    a.count = const_cast<int32_t *>(count); a.out = out; a.lse = lse; a.status = status;
    switch (Hq / Hkv) {
        case 1: return launch_gather_cluster_g<1>(a, B, st);
        case 2: return launch_gather_cluster_g<2>(a, B, st);
        case 4: return launch_gather_cluster_g<4>(a, B, st);
        case 8: return launch_gather_cluster_g<8>(a, B, st);
        default: return cudaErrorInvalidValue;
    }
}

template <int G, int S, int CS>
static void fused_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute (&attr)[2], int Hkv, int B, cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(CS, Hkv, B);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = fused_smem_bytes(G, S, CS);
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
}

// Opt in to the shared-memory carve-out (once per device) and return how many clusters of this variant the
// device holds at once (0 on error).
template <int G, int S, int CS, bool kHost = false>
static int fused_prepare() {
    static int clusters[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!clusters[dev]) {
        if (cudaFuncSetAttribute(fused_step_kernel<G, S, CS, kHost>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 fused_smem_bytes(G, S, CS)) != cudaSuccess)
            return 0;
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[2];
        fused_config<G, S, CS>(cfg, attr, 1, 64, nullptr);
        cfg.numAttrs = 1;   // the cluster shape is all the occupancy query looks at
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, fused_step_kernel<G, S, CS, kHost>, &cfg) != cudaSuccess || n <= 0) return 0;
        clusters[dev] = n;
    }
    return clusters[dev];
}

template <int G, int S, int CS, bool kHost = false>
static cudaError_t launch_fused_gsc(const FusedArgs &args, int B, cudaStream_t st) {
    if (fused_prepare<G, S, CS, kHost>() <= 0) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    fused_config<G, S, CS>(cfg, attr, args.Hkv, B, st);
    cudaError_t e = cudaLaunchKernelEx(&cfg, fused_step_kernel<G, S, CS, kHost>, args);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

// Variant for a step of `units` (sequence, KV head) pairs with index lists of up to k_max entries: the number
// of row stages per warp in *stages, the cluster size as the result, 0 if the step does not fit (a
// cluster that had to wait for another one to finish would double the latency).
//  * lists of up to 1024 entries (one block per warp with clusters of 8): the one-stage kernel, two CTAs per
//    SM, with the larger cluster, 8 or 4 CTAs per unit, of which `units` are resident at once;
//  * longer lists: the two-stage kernel (one CTA per SM, clusters of 8) while `units` of its clusters are
//    resident at once, else, up to kFusedOneStageMaxK entries, the one-stage kernel as above (its warps then
//    take their blocks one after the other).
// Clusters of 2 work as well (the kernel is written for them) but lose to the three-kernel path at the batch
// sizes they would serve (45.7 against 41.3 us at 128 units), so they are not offered.
template <int G>
static int fused_variant(long long units, int k_max, int *stages) {
    const bool one_block_per_warp = k_max <= kFusedMaxCS * kFusedWarps * kBlockTokens;
    if (!one_block_per_warp && units <= fused_prepare<G, 2, 8>()) {
        *stages = 2;
        return 8;
    }
    *stages = 1;
    if (k_max > kFusedOneStageMaxK) return 0;
    if (units <= fused_prepare<G, 1, 8>()) return 8;
    if (units <= fused_prepare<G, 1, 4>()) return 4;
    return 0;
}

bool fused_step_eligible(int B, int Hq, int Hkv, int max_seq_len, int k_max) {
    if (max_seq_len > kFusedMaxSeq || Hkv <= 0) return false;
    const long long units = (long long)B * Hkv;
    int stages = 0;
    switch (Hq / Hkv) {
        case 1: return fused_variant<1>(units, k_max, &stages) > 0;
        case 2: return fused_variant<2>(units, k_max, &stages) > 0;
        case 4: return fused_variant<4>(units, k_max, &stages) > 0;
        case 8: return fused_variant<8>(units, k_max, &stages) > 0;
        default: return false;
    }
}

bool fused_step_from_host_eligible(int B, int Hq, int Hkv, int max_seq_len, int k_max) {
    if (max_seq_len > kFusedMaxSeq || Hkv <= 0) return false;
    const long long units = (long long)B * Hkv;
    int stages = 0, cs = 0;
    switch (Hq / Hkv) {
        case 1: cs = fused_variant<1>(units, k_max, &stages); break;
        case 2: cs = fused_variant<2>(units, k_max, &stages); break;
        case 4: cs = fused_variant<4>(units, k_max, &stages); break;
        case 8: cs = fused_variant<8>(units, k_max, &stages); break;
        default: return false;
    }
    return cs > 0 && stages == 1;
}

template <int G>
static cudaError_t launch_fused_g(const FusedArgs &args, int B, cudaStream_t st) {
    int stages = 0;
    const int cs = fused_variant<G>((long long)B * args.Hkv, args.k_max, &stages);
    if (args.v_new) {   // host-buffer entry: only the one-stage variants read their inputs across the bus
        if (stages == 1 && cs == 8) return launch_fused_gsc<G, 1, 8, true>(args, B, st);
        if (stages == 1 && cs == 4) return launch_fused_gsc<G, 1, 4, true>(args, B, st);
        return cudaErrorInvalidConfiguration;
    }
    if (stages == 2 && cs == 8) return launch_fused_gsc<G, 2, 8>(args, B, st);
    if (cs == 8) return launch_fused_gsc<G, 1, 8>(args, B, st);
    if (cs == 4) return launch_fused_gsc<G, 1, 4>(args, B, st);
    return cudaErrorInvalidConfiguration;
}

cudaError_t launch_fused_step(int B, int Hq, int Hkv, float sm_scale, const MapView &map_q, const MapView &map_k,
                              const uint16_t *q, const uint16_t *k_new, TensorView K, TensorView V, uint32_t *k_codes,
                              long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq,
                              int k_uniform, int max_seq_len, int k_max, uint32_t *q_codes, int32_t *idx,
                              long long idx_sb, long long idx_sh, int32_t *count, uint16_t *out, float *lse,
                              cudaStream_t st, Windows win, const int32_t *block_table, long long bt_sb, int page_shift,
                              const uint16_t *v_new_host) {
    FusedArgs a{};
    a.v_new = v_new_host;
    a.win = win;
    a.block_table = block_table; a.bt_sb = bt_sb; a.page_shift = page_shift;
    a.page_rows = (block_table && K.sn > 0) ? (int)(K.sb / K.sn) : 0;
    a.map_q = map_q; a.map_k = map_k; a.q = q; a.k_new = k_new; a.K = K; a.V = V;
    a.k_codes = k_codes; a.kc_sb = kc_sb; a.kc_sh = kc_sh; a.seq_lens = seq_lens; a.k_per_seq = k_per_seq;
    a.k_uniform = k_uniform; a.max_seq_len = max_seq_len; a.k_max = k_max; a.Hq = Hq; a.Hkv = Hkv;
    a.scale_log2 = sm_scale * kLog2e; a.q_codes = q_codes; a.idx = idx; a.idx_sb = idx_sb; a.idx_sh = idx_sh;
    a.count = count; a.out = out; a.lse = lse;
    switch (Hq / Hkv) {
        case 1: return launch_fused_g<1>(a, B, st);
        case 2: return launch_fused_g<2>(a, B, st);
        case 4: return launch_fused_g<4>(a, B, st);
        case 8: return launch_fused_g<8>(a, B, st);
        default: return cudaErrorInvalidValue;
    }
}

} // namespace ha
