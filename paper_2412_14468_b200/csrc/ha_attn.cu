// GATHER-ATT (Section 4) and dense single-query SDPA (Section 3.1) as one persistent split-K
// flash-decode kernel.  The 256-byte bf16 K/V rows are read in place through the indices
// (Section 4.4: no gather into a buffer) and every row is read from HBM once for all G query heads
// of its KV head.
//
// Scheduling.  The index lists of all (sequence, KV head) units are cut into blocks of 16 entries;
// the blocks of all units, laid end to end, are divided evenly over a fixed number of CTAs (two per
// SM), whatever the batch size and however ragged the lists are.  A CTA walks its range unit by
// unit; where a unit is shared by several CTAs each publishes its running (max, sum, output) state
// and the CTA that arrives last (a ticket counter; nobody waits) merges them, normalises and
// rounds once to bf16.
//
// Data path per warp: a private ring in shared memory holds kStages blocks of rows; rows are
// fetched with 16-byte cp.async (a half-warp per 256-byte row) two blocks ahead of their use, the
// list entries one block further ahead.  S[head][token] = Q K^T and O^T[d][head] += V^T P^T run on
// the tensor cores from ldmatrix fragments (mma.sync m16n8k16, bf16 in, fp32 accumulate; P is
// split into bf16 hi + lo parts so the weights keep ~16 bits), softmax online in fp32 in the log2
// domain.  At ~4 FLOP/B the kernel is bound by HBM; the tensor cores only keep the instruction
// count out of the way.
#include <atomic>
#include "ha_attn_dev.cuh"

namespace ha {

constexpr int kAttnWarps = 4;
constexpr int kAttnThreads = kAttnWarps * 32;
constexpr int kStages = 3;                    // blocks of rows in flight per warp (ring in shared memory)
constexpr int kWarpRingBytes = kStages * kStageBytes;
constexpr int kAttnSmemBytes = kAttnWarps * kWarpRingBytes;

struct AttnArgs {
    const uint16_t *q;
    TensorView K, V;
    const int32_t *seq_lens, *idx, *count;
    long long idx_sb, idx_sh;
    const int32_t *k_per_seq;   // with count_from_k: budget per sequence (or NULL: k_uniform)
    int k_uniform, count_from_k;
    Windows win;                // with count_from_k: tokens always kept in addition to the budget
    // paged K/V (block_table != NULL): token t of sequence b lives in page block_table[b*bt_sb + (t >> page_shift)],
    // slot t & (2^page_shift - 1); K.sb / V.sb are then the page strides and page_rows = K.sb / K.sn
    const int32_t *block_table;
    long long bt_sb;
    int page_shift, page_rows;
    int max_items, Hq, Hkv, n_units, balanced;
    int kv_shift;               // unit head h reads K/V head h >> kv_shift (0 unless every query head has its own list)
    float scale_log2;
    float *part_ml, *part_acc;
    int32_t *tickets;
    uint32_t *status;
    uint16_t *out;
    float *lse;
};

template <int G, bool kGather>
__global__ void __launch_bounds__(kAttnThreads, 2) attn_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char ring[];   // kAttnWarps private rings, then the block prefix
    __shared__ float s_m[kAttnWarps][8], s_l[kAttnWarps][8];
    __shared__ uint32_t s_mask[kAttnWarps][kStages];
    __shared__ int s_last;
    int *s_pref = reinterpret_cast<int *>(ring + kAttnSmemBytes);   // [n_units + 1] in balanced mode

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int cta = blockIdx.x, P = gridDim.x;
    const int Hq = a.Hq, Hkv = a.Hkv;
    unsigned char *my_ring = ring + warp * kWarpRingBytes;
    const uint32_t ring_u32 = smem_u32(my_ring);
    bool bad = false;

    // The index lists and the appended rows come from the preceding kernels: they are read after the
    // programmatic-launch wait.  Inside a whole layer-step the list LENGTHS are min(k, n) by
    // construction, so the work distribution is computed before the wait, from inputs that no kernel
    // of the step writes; a stand-alone call reads the caller's count array instead, after the wait.
    pdl_launch_dependents();
    const bool early = kGather ? (a.count_from_k != 0) : true;
    if (!early) pdl_wait();

    auto unit_count = [&](int u) -> int {
        const int b = u / Hkv;
        const int n_b = a.seq_lens[b];
        int c = n_b;
        if (kGather) {
            if (a.count_from_k) {   // what SCORE + TOPK is about to report: windows plus the budget among the others
                const int nf = forced_before(window_bounds(a.win, max(n_b, 0)), max(n_b, 0));
                const int kb = a.k_per_seq ? a.k_per_seq[b] : a.k_uniform;
                c = nf + max(0, min(min(kb, a.max_items - nf), n_b - nf));
            } else {
                c = a.count[u];
            }
        }
        return max(0, min(c, a.max_items));
    };
    auto write_empty = [&](int u) {   // empty selection: out = 0, lse = -inf
        const long long h0 = (long long)(u / Hkv) * Hq + (long long)(u % Hkv) * G;
        for (int i = tid; i < G * kD; i += kAttnThreads) a.out[h0 * kD + i] = 0;
        if (a.lse && tid < G) a.lse[h0 + tid] = -CUDART_INF_F;
    };

    // ---- this CTA's range [x, x_end) of the global block sequence
    long long x, x_end, T, Pe = P;   // Pe: CTAs that take part in the split
    int u;
    if (a.balanced) {
        if (a.n_units <= 32) {
            // few units: every warp scans the block counts in registers (no barrier); warp 0 keeps a copy
            const int nb = (lane < a.n_units) ? (unit_count(lane) + kBlockTokens - 1) / kBlockTokens : 0;
            int inc = nb;
#pragma unroll
            for (int dd = 1; dd < 32; dd <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, inc, dd);
                if (lane >= dd) inc += o;
            }
            if (warp == 0) {
                if (lane == 0) s_pref[0] = 0;
                if (lane < a.n_units) s_pref[lane + 1] = inc;
            }
            __syncthreads();
        } else {
            for (int v = tid; v < a.n_units; v += kAttnThreads)
                s_pref[v + 1] = (unit_count(v) + kBlockTokens - 1) / kBlockTokens;
            if (tid == 0) s_pref[0] = 0;
            __syncthreads();
            if (warp == 0) {   // inclusive scan in place, one contiguous piece per lane
                const int per = (a.n_units + 31) / 32;
                const int lo = min(a.n_units, lane * per), hi = min(a.n_units, lo + per);
                int sum = 0;
                for (int v = lo; v < hi; ++v) sum += s_pref[v + 1];
                int inc = sum;
#pragma unroll
                for (int dd = 1; dd < 32; dd <<= 1) {
                    const int o = __shfl_up_sync(0xffffffffu, inc, dd);
                    if (lane >= dd) inc += o;
                }
                int run = inc - sum;
                for (int v = lo; v < hi; ++v) { run += s_pref[v + 1]; s_pref[v + 1] = run; }
            }
            __syncthreads();
        }
        T = s_pref[a.n_units];
        // Fewer blocks than CTAs (lists much shorter than the rows that hold them): only the first T CTAs take a
        // range, one block each.  With the full grid in the formulas some CTAs of a unit's range would be empty
        // and leave without a ticket, and the unit would never be finalised.
        if (T > 0 && T < Pe) Pe = T;
        // Lists of equal length and at least three units per four CTAs: one whole unit per CTA and the other CTAs
        // idle.  Cutting every unit across two CTAs costs each of them a second prologue, a drained row pipeline
        // and a merge through global memory, which is more than the idle slots are worth (256 units on 296 CTAs:
        // 29.7 against 34.7 us).  The lengths are only known here, so the choice is made on the device.
        if (a.n_units > 32 && a.n_units <= P && a.n_units * 4 >= P * 3) {   // CTA-uniform
            const int nb0 = s_pref[1];
            bool same = nb0 > 0;
            for (int v = tid; v < a.n_units; v += kAttnThreads) same = same && (s_pref[v + 1] - s_pref[v] == nb0);
            if (__syncthreads_and(same)) Pe = a.n_units;
        }
        x = (T > 0 && cta < Pe) ? (long long)cta * T / Pe : 0;
        x_end = (T > 0 && cta < Pe) ? (long long)(cta + 1) * T / Pe : 0;
        int lo = 0, hi = a.n_units;   // largest u with s_pref[u] <= x
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_pref[mid] <= x) lo = mid; else hi = mid;
        }
        u = lo;
    } else {   // one CTA per unit
        u = cta;
        T = 0;
        x = 0;
        x_end = (unit_count(u) + kBlockTokens - 1) / kBlockTokens;
    }
    if (early) pdl_wait();   // nothing is written, and nothing of the preceding kernels read, before this point
    if (a.balanced) {
        for (int v = cta; v < a.n_units; v += P)
            if (s_pref[v + 1] == s_pref[v]) write_empty(v);
    } else if (x_end == 0) {
        write_empty(u);
    }
    if (x >= x_end) return;

    while (x < x_end) {
        // ---- segment: blocks [blk_lo, blk_hi) of unit u
        long long u_lo = 0, u_hi = x_end;
        int n_parts = 1, my_part = 0, slot0 = 0;
        if (a.balanced) {
            u_lo = s_pref[u];
            u_hi = s_pref[u + 1];
            const int c_first = (int)(((u_lo + 1) * Pe - 1) / T), c_last = (int)((u_hi * Pe - 1) / T);
            n_parts = c_last - c_first + 1;
            my_part = cta - c_first;
            slot0 = c_first + u;   // slots of a unit are consecutive: CTA index + unit index
        }
        const long long seg_end = (x_end < u_hi) ? x_end : u_hi;
        const int blk_lo = (int)(x - u_lo), blk_hi = (int)(seg_end - u_lo);
        const int b = u / Hkv, kvh = u % Hkv;
        const int n = a.seq_lens[b];
        const int cnt = unit_count(u);
        const long long head0 = (long long)b * Hq + (long long)kvh * G;
        const int start = blk_lo * kBlockTokens, end = min(cnt, blk_hi * kBlockTokens);

        const bool paged = kGather && a.block_table != nullptr;   // rows are then addressed from the pool's base
        const unsigned char *Kb = reinterpret_cast<const unsigned char *>(a.K.ptr + (paged ? 0LL : (long long)b * a.K.sb) + (long long)(kvh >> a.kv_shift) * a.K.sh);
        const unsigned char *Vb = reinterpret_cast<const unsigned char *>(a.V.ptr + (paged ? 0LL : (long long)b * a.V.sb) + (long long)(kvh >> a.kv_shift) * a.V.sh);
        const int32_t *pages = paged ? a.block_table + (long long)b * a.bt_sb : nullptr;
        const long long k_row = a.K.sn * 2, v_row = a.V.sn * 2;   // bytes
        const int32_t *list = kGather ? a.idx + (long long)b * a.idx_sb + (long long)kvh * a.idx_sh : nullptr;

        // raw list entry of position p for this lane; only the load is issued here, the value is first
        // looked at when its block is started, one iteration later, so the warp never waits on it
        auto fetch_raw = [&](int p) -> int { return (kGather && p < end) ? __ldg(list + p) : p; };
        // row to fetch for a raw entry (-1: past the slice, padding or outside the sequence).  Contiguous cache:
        // the token id itself; paged cache: page * rows per page stride + slot, which costs one more load,
        // so rows are resolved one block before they are requested and list entries one block before that.
        auto row_of = [&](int p, int raw) -> int {
            int t = (p < end) ? raw : -1;
            if (t >= n) { bad = true; t = -1; }
            if (paged && t >= 0) t = __ldg(pages + (t >> a.page_shift)) * a.page_rows + (t & ((1 << a.page_shift) - 1));
            return t;
        };
        auto issue = [&](int stg, int my_t) {
            const uint32_t valid = attn_issue_block(ring_u32 + stg * kStageBytes, Kb, Vb, k_row, v_row, my_t, lane);
            if (lane == 0) s_mask[warp][stg] = valid;
        };

        // ---- software pipeline over this warp's blocks: block i lives at first + i * stride
        const int stride = kAttnWarps * kBlockTokens;
        const int first = start + warp * kBlockTokens;
        const int nblk = (first < end) ? (end - first + stride - 1) / stride : 0;
        int raw[kStages + 1];
#pragma unroll
        for (int i = 0; i < kStages + 1; ++i) raw[i] = fetch_raw(first + i * stride + (lane & 15));

        uint32_t qa[8][2];
        attn_load_q<G>(qa, a.q + head0 * kD, lane);
        float acc[8][4];
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
        float m_run = -CUDART_INF_F, l_run = 0.0f;

#pragma unroll
        for (int i = 0; i < kStages - 1; ++i) {
            if (i < nblk) issue(i, row_of(first + i * stride + (lane & 15), raw[i]));
            cp_async_commit();
        }
        int next_row = row_of(first + (kStages - 1) * stride + (lane & 15), raw[kStages - 1]);   // row of block kStages-1
        int after_raw = raw[kStages];                                                            // list entry of the block after it
        int st = 0;
        for (int i = 0; i < nblk; ++i) {
            {   // refill the stage that block i-1 just released
                const int j = i + kStages - 1;
                const int pj = first + j * stride;
                int stj = st + kStages - 1;
                if (stj >= kStages) stj -= kStages;
                if (j < nblk) issue(stj, next_row);
                cp_async_commit();
                next_row = row_of(pj + stride + (lane & 15), after_raw);      // one block ahead
                after_raw = fetch_raw(pj + 2 * stride + (lane & 15));         // two blocks ahead
            }
            cp_async_wait<kStages - 1>();
            __syncwarp();
            const uint32_t valid = s_mask[warp][st];
            const uint32_t ks = ring_u32 + st * kStageBytes;
            const uint32_t vs = ks + kTileBytes;
            attn_consume_block(ks, vs, valid, qa, a.scale_log2, lane, acc, m_run, l_run);
            __syncwarp();   // every lane is done with this stage before it is refilled
            if (++st == kStages) st = 0;
        }
        cp_async_wait<0>();

        // ---- merge the warps of this CTA through shared memory (each warp reuses its own ring)
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        if (c == 0) { s_m[warp][g] = m_run; s_l[warp][g] = l_run; }
        __syncwarp();
        float *my_acc = reinterpret_cast<float *>(my_ring);   // [G][128]
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int h = 2 * c + hh;
            if (h < G) {
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    my_acc[h * kD + 16 * mt + g] = acc[mt][hh];
                    my_acc[h * kD + 16 * mt + 8 + g] = acc[mt][2 + hh];
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
                    A = fmaf(reinterpret_cast<const float *>(ring + w * kWarpRingBytes)[j * kD + d], f, A);
                }
            }
            Mj[j] = M; Lj[j] = L; Aj[j] = A;
        }

        bool finalize = true;
        if (n_parts > 1) {
            // publish this part, take a ticket; the CTA that draws the last ticket merges all parts
            const long long slot = (long long)(slot0 + my_part) * G;
#pragma unroll
            for (int j = 0; j < G; ++j) {
                a.part_acc[(slot + j) * kD + d] = Aj[j];
                if (d == 0) { a.part_ml[(slot + j) * 2] = Mj[j]; a.part_ml[(slot + j) * 2 + 1] = Lj[j]; }
            }
            __threadfence();
            __syncthreads();
            if (tid == 0) {
                const int t = atomicAdd(&a.tickets[u], 1);
                s_last = (t == n_parts - 1);
                if (s_last) a.tickets[u] = 0;   // ready for the next call
            }
            __syncthreads();
            finalize = (s_last != 0);
            if (finalize) {
                __threadfence();
                // Merge of the parts: thread (dq, pg) owns dimensions 4dq..4dq+3 and the parts pg, pg+4, ...;
                // a pass covers 16 (8 when G = 8) parts with every load issued before the first use (one L2 round trip),
                // then the four part groups are folded through shared memory.
                const int dq = tid & 31, pg = tid >> 5;
                float Mt[G], Lt[G];
                float4 At[G];
#pragma unroll
                for (int j = 0; j < G; ++j) { Mt[j] = -CUDART_INF_F; Lt[j] = 0.0f; At[j] = make_float4(0.f, 0.f, 0.f, 0.f); }
                constexpr int kEB = (G >= 8) ? 2 : 4;   // loads in flight per head and thread
                for (int part0 = 0; part0 < n_parts; part0 += 4 * kEB) {
                    float4 av[G][kEB];
                    float mv[G][kEB], lv[G][kEB];
#pragma unroll
                    for (int e = 0; e < kEB; ++e) {
                        const int pp = part0 + 4 * e + pg;
                        const bool ok = pp < n_parts;
#pragma unroll
                        for (int j = 0; j < G; ++j) {
                            const long long sl = (long long)(slot0 + (ok ? pp : 0)) * G + j;
                            const float2 ml = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + sl * 2));
                            av[j][e] = __ldcg(reinterpret_cast<const float4 *>(a.part_acc + sl * kD) + dq);
                            mv[j][e] = ok ? ml.x : -CUDART_INF_F;
                            lv[j][e] = ok ? ml.y : 0.0f;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < G; ++j) {
                        float M = Mt[j];
#pragma unroll
                        for (int e = 0; e < kEB; ++e) M = fmaxf(M, mv[j][e]);
                        if (M > -CUDART_INF_F) {
                            const float f0 = exp2f(Mt[j] - M);
                            float L = Lt[j] * f0;
                            float4 A = make_float4(At[j].x * f0, At[j].y * f0, At[j].z * f0, At[j].w * f0);
#pragma unroll
                            for (int e = 0; e < kEB; ++e) {
                                const float f = exp2f(mv[j][e] - M);   // 0 for absent parts
                                L = fmaf(lv[j][e], f, L);
                                A.x = fmaf(av[j][e].x, f, A.x); A.y = fmaf(av[j][e].y, f, A.y);
                                A.z = fmaf(av[j][e].z, f, A.z); A.w = fmaf(av[j][e].w, f, A.w);
                            }
                            Mt[j] = M; Lt[j] = L; At[j] = A;
                        }
                    }
                }
                __syncthreads();   // the rings were last read by the warp merge above
                float *red = reinterpret_cast<float *>(ring);   // [4 part groups][G][128] + [4][G][2]
                float *red_ml = red + kAttnWarps * G * kD;
#pragma unroll
                for (int j = 0; j < G; ++j) {
                    reinterpret_cast<float4 *>(red + (pg * G + j) * kD)[dq] = At[j];
                    if (dq == 0) { red_ml[(pg * G + j) * 2] = Mt[j]; red_ml[(pg * G + j) * 2 + 1] = Lt[j]; }
                }
                __syncthreads();
#pragma unroll
                for (int j = 0; j < G; ++j) {
                    float M = -CUDART_INF_F;
#pragma unroll
                    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, red_ml[(w * G + j) * 2]);
                    float L = 0.0f, A = 0.0f;
                    if (M > -CUDART_INF_F) {
#pragma unroll
                        for (int w = 0; w < kAttnWarps; ++w) {
                            const float f = exp2f(red_ml[(w * G + j) * 2] - M);
                            L = fmaf(red_ml[(w * G + j) * 2 + 1], f, L);
                            A = fmaf(red[(w * G + j) * kD + d], f, A);
                        }
                    }
                    Mj[j] = M; Lj[j] = L; Aj[j] = A;
                }
            }
        }
        if (finalize) {
#pragma unroll
            for (int j = 0; j < G; ++j) {
                const float o = (Lj[j] > 0.0f) ? Aj[j] / Lj[j] : 0.0f;
                const __nv_bfloat16 ob = __float2bfloat16_rn(o);
                a.out[(head0 + j) * kD + d] = *reinterpret_cast<const uint16_t *>(&ob);
                if (a.lse && d == 0) a.lse[head0 + j] = (Lj[j] > 0.0f) ? (Mj[j] * kLn2 + logf(Lj[j])) : -CUDART_INF_F;
            }
        }

        // ---- next unit of this CTA's range (units without blocks are skipped)
        x = seg_end;
        if (x < x_end) {
            ++u;
            while (s_pref[u + 1] == s_pref[u]) ++u;
            __syncthreads();   // the rings are reused by the next segment
        }
    }
    if (bad) atomicOr(a.status, HA_DEV_BAD_INDEX);
}

template <int G, bool kGather>
static cudaError_t launch_attn_t(const AttnArgs &args, int grid, size_t smem, cudaStream_t st) {
    static bool done[64] = {};   // opt in to the ring's shared memory once per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(attn_kernel<G, kGather>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kAttnSmemBytes + (kMaxBalancedUnits + 1) * 4);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    cudaError_t e = launch_pdl(attn_kernel<G, kGather>, dim3(grid), dim3(kAttnThreads), smem, st, args);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

template <int G>
static cudaError_t launch_attn_g(bool gather, const AttnArgs &args_in, cudaStream_t st) {
    AttnArgs args = args_in;
    const long long blocks_per_unit = (args.max_items + kBlockTokens - 1) / kBlockTokens;
    const long long t_max = blocks_per_unit * args.n_units;
    int grid;
    size_t smem = kAttnSmemBytes;
    if (args.n_units <= kMaxBalancedUnits) {
        args.balanced = 1;
        long long want = (t_max + kAttnWarps - 1) / kAttnWarps;   // at least one block per warp
        const long long cap = (long long)min(2 * sm_count(), kMaxAttnCtas);
        grid = (int)max(1LL, min(want, cap));
        // a CTA count that is a multiple of the unit count lets equal-length lists split at CTA borders,
        // so that no CTA pays a second prologue and merge in the middle of its range; with fewer than two CTAs
        // per unit the rounding would only leave CTA slots empty (256 ragged units: 296 CTAs, 54.9 against 56.7 us)
        if (args.n_units * 2 <= grid) grid = grid / args.n_units * args.n_units;
        else if (args.n_units > grid) {
            // more units than CTAs: m whole units per CTA (no unit is split, so nothing is published and
            // merged through global memory) when that still fills most of the CTA slots (measured at 512 equal units:
            // 256 CTAs with two whole units each beat 296 CTAs with split units, 54.0 against 55.9 us)
            const int m = (args.n_units + grid - 1) / grid;
            if (args.n_units % m == 0 && (long long)(args.n_units / m) * 5 >= (long long)grid * 4) grid = args.n_units / m;
        }
        smem += (size_t)(args.n_units + 1) * 4;
    } else {
        args.balanced = 0;
        grid = args.n_units;
    }
    return gather ? launch_attn_t<G, true>(args, grid, smem, st) : launch_attn_t<G, false>(args, grid, smem, st);
}

cudaError_t launch_attention(bool gather, int B, int Hq, int Hkv, float sm_scale, const uint16_t *q,
                             TensorView K, TensorView V, const int32_t *seq_lens, const int32_t *idx,
                             long long idx_sb, long long idx_sh, const int32_t *count, int max_items,
                             uint16_t *out, float *lse, float *part_ml, float *part_acc, int32_t *tickets,
                             uint32_t *status, cudaStream_t st, int count_from_k, const int32_t *k_per_seq,
                             int k_uniform, Windows win, const int32_t *block_table, long long bt_sb, int page_shift,
                             int kv_shift) {
    AttnArgs a{};
    a.kv_shift = kv_shift;
    a.win = win;
    a.block_table = block_table; a.bt_sb = bt_sb; a.page_shift = page_shift;
    a.page_rows = (block_table && K.sn > 0) ? (int)(K.sb / K.sn) : 0;
    a.q = q; a.K = K; a.V = V; a.seq_lens = seq_lens; a.idx = idx; a.count = count;
    a.idx_sb = idx_sb; a.idx_sh = idx_sh; a.max_items = max_items; a.Hq = Hq; a.Hkv = Hkv;
    a.n_units = B * Hkv; a.scale_log2 = sm_scale * kLog2e;
    a.k_per_seq = k_per_seq; a.k_uniform = k_uniform; a.count_from_k = count_from_k;
    a.part_ml = part_ml; a.part_acc = part_acc; a.tickets = tickets; a.status = status; a.out = out; a.lse = lse;
    switch (Hq / Hkv) {
        case 1: return launch_attn_g<1>(gather, a, st);
        case 2: return launch_attn_g<2>(gather, a, st);
        case 4: return launch_attn_g<4>(gather, a, st);
        case 8: return launch_attn_g<8>(gather, a, st);
        default: return cudaErrorInvalidValue;
    }
}

// Host-driven entry only: writes this step's new K and V rows into the cache at slot seq_len-1 and,
// if q_src is given, copies the query vectors into the device staging buffer.  The sources may be
// device memory or pinned host memory mapped into the device's address space (then this kernel IS
// the host-to-device transfer: one launch instead of three copy operations).
__global__ void append_kv_kernel(int Hq, int Hkv, const uint16_t *__restrict__ k_new,
                                 const uint16_t *__restrict__ v_new, TensorView K, TensorView V,
                                 const int32_t *__restrict__ seq_lens, const uint16_t *__restrict__ q_src,
                                 uint16_t *__restrict__ q_dst, uint16_t *__restrict__ k_dst,
                                 const int32_t *__restrict__ block_table, long long bt_sb, int page_shift, int page_rows) {
    const int g = blockIdx.x, b = blockIdx.y, t = threadIdx.x;   // 32 threads x 8 bytes per row
    const long long src = ((long long)b * Hkv + g) * kD;
    const uint2 kv = reinterpret_cast<const uint2 *>(k_new + src)[t];
    const uint2 vv = reinterpret_cast<const uint2 *>(v_new + src)[t];
    if (k_dst) reinterpret_cast<uint2 *>(k_dst + src)[t] = kv;   // device copy of k_new for ENCODE
    if (q_src) {
        const int G = Hq / Hkv;
        for (int j = 0; j < G; ++j) {
            const long long qo = ((long long)b * Hq + (long long)g * G + j) * kD;
            reinterpret_cast<uint2 *>(q_dst + qo)[t] = reinterpret_cast<const uint2 *>(q_src + qo)[t];
        }
    }
    const int slot = seq_lens[b] - 1;
    if (slot < 0) return;
    // contiguous cache: row `slot` of sequence b; paged cache: the row of the pool that the block table names
    long long base_b = b, row = slot;
    if (block_table) {
        base_b = 0;
        row = (long long)block_table[(long long)b * bt_sb + (slot >> page_shift)] * page_rows + (slot & ((1 << page_shift) - 1));
    }
    uint16_t *kd = const_cast<uint16_t *>(K.ptr) + base_b * K.sb + (long long)g * K.sh + row * K.sn;
    uint16_t *vd = const_cast<uint16_t *>(V.ptr) + base_b * V.sb + (long long)g * V.sh + row * V.sn;
    reinterpret_cast<uint2 *>(kd)[t] = kv;
    reinterpret_cast<uint2 *>(vd)[t] = vv;
}

cudaError_t launch_append_kv(int B, int Hq, int Hkv, const uint16_t *k_new, const uint16_t *v_new, TensorView K,
                             TensorView V, const int32_t *seq_lens, const uint16_t *q_src, uint16_t *q_dst,
                             uint16_t *k_dst, cudaStream_t st, const int32_t *block_table, long long bt_sb, int page_shift) {
    const int page_rows = (block_table && K.sn > 0) ? (int)(K.sb / K.sn) : 0;
    append_kv_kernel<<<dim3(Hkv, B), 32, 0, st>>>(Hq, Hkv, k_new, v_new, K, V, seq_lens, q_src, q_dst, k_dst, block_table,
                                                  bt_sb, page_shift, page_rows);
    count_launch();
    return cudaGetLastError();
}

} // namespace ha

// ------------------------------------------------------------------ entry point with built-in scratch
//
// ha_gather_attn_static: GATHER-ATT for callers that cannot hand the library a workspace because
// they cannot allocate device memory themselves (see include/hashattn.h).  The split-K states, the
// ticket counters and the status word live in the file-scope array below, which every GPU that
// loads the library carries until the process exits.

namespace ha {
constexpr int kStaticMaxUnits = 64;     // (sequence, KV head) pairs
constexpr int kStaticMaxCtas = 512;     // persistent CTAs (2 per SM) the scratch has room for
constexpr size_t kStaticSlots = (size_t)kStaticMaxCtas + kStaticMaxUnits;
constexpr size_t kStaticTicketsOff = 256;                                    // after the status word
constexpr size_t kStaticMlOff = kStaticTicketsOff + 256;                     // 64 counters x 4 bytes
constexpr size_t kStaticAccOff = kStaticMlOff + ((kStaticSlots * kMaxGroup * 2 * 4 + 255) / 256) * 256;
constexpr size_t kStaticBytes = kStaticAccOff + kStaticSlots * kMaxGroup * kD * 4;   // about 2.4 MB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];
} // namespace ha

extern "C" int ha_gather_attn_static(const ha_shape *shape, const uint16_t *q, const ha_tensor *K, const ha_tensor *V,
                                     const int32_t *seq_lens, const int32_t *idx, int64_t idx_stride_b,
                                     int64_t idx_stride_h, const int32_t *count, int32_t k_max, uint16_t *out,
                                     float *lse, void *stream) {
    using namespace ha;
    if (!shape || !q || !K || !V || !K->ptr || !V->ptr || !seq_lens || !idx || !count || !out || k_max < 0)
        return HA_ERR_INVALID_ARG;
    if (shape->batch < 0 || shape->n_q_heads <= 0 || shape->n_kv_heads <= 0) return HA_ERR_INVALID_ARG;
    if (shape->head_dim != kD || shape->n_q_heads % shape->n_kv_heads != 0) return HA_ERR_UNSUPPORTED;
    const int G = shape->n_q_heads / shape->n_kv_heads;
    if (G != 1 && G != 2 && G != 4 && G != 8) return HA_ERR_UNSUPPORTED;
    if (((uintptr_t)q & 15) || ((uintptr_t)K->ptr & 15) || ((uintptr_t)V->ptr & 15) || (K->stride_b & 7) ||
        (K->stride_h & 7) || (K->stride_n & 7) || (V->stride_b & 7) || (V->stride_h & 7) || (V->stride_n & 7) ||
        K->stride_n < kD || V->stride_n < kD)
        return HA_ERR_INVALID_ARG;
    // the built-in scratch is sized for at most kStaticMaxUnits units and kStaticMaxCtas CTAs
    if ((long long)shape->batch * shape->n_kv_heads > kStaticMaxUnits) return HA_ERR_STATIC_LIMIT;
    if (2 * sm_count() > kStaticMaxCtas) return HA_ERR_STATIC_LIMIT;
    if (shape->batch == 0) return HA_OK;

    // Set-up, once per device: in host code the array's name is only a stand-in for the symbol; the
    // device address that a kernel can use has to be asked for, with the device current.
    static std::atomic<void *> scratch_of_device[64];   // zero-initialised; two threads that race store the same address
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HA_ERR_CUDA;
    void *scratch = scratch_of_device[dev].load(std::memory_order_acquire);
    if (!scratch) {
        if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) return HA_ERR_CUDA;
        scratch_of_device[dev].store(scratch, std::memory_order_release);
    }
    unsigned char *base = reinterpret_cast<unsigned char *>(scratch);
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the last call left: the status word and the ticket counters must start at zero
    if (cudaMemsetAsync(base, 0, kStaticMlOff, st) != cudaSuccess) return HA_ERR_CUDA;
    TensorView Kv{reinterpret_cast<const uint16_t *>(K->ptr), (long long)K->stride_b, (long long)K->stride_h,
                  (long long)K->stride_n};
    TensorView Vv{reinterpret_cast<const uint16_t *>(V->ptr), (long long)V->stride_b, (long long)V->stride_h,
                  (long long)V->stride_n};
    if (launch_attention(true, shape->batch, shape->n_q_heads, shape->n_kv_heads, shape->sm_scale, q, Kv, Vv, seq_lens,
                         idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                         reinterpret_cast<float *>(base + kStaticMlOff), reinterpret_cast<float *>(base + kStaticAccOff),
                         reinterpret_cast<int32_t *>(base + kStaticTicketsOff), reinterpret_cast<uint32_t *>(base),
                         st) != cudaSuccess)
        return HA_ERR_CUDA;
    return HA_OK;
}

