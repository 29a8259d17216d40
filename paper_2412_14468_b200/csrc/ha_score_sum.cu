// SCORE + TOPK with the per-head scores of a GQA group ADDED instead of maximised: S(i) = sum over the G query
// heads of (32 - popc(k_i xor q_j)) (Eq. 1 with the bitcount identity of Section 4.1, per head), 0 .. 32 G, then the
// standard top-k of Section 4 with ties towards the lowest token index.  The paper defines the score for one query
// head; the layer-step reduces a group with the maximum (33 levels), this is the stand-alone alternative with
// 32 G + 1 levels.
//
// One thread-block cluster (1 to 16 CTAs, by the number of units) per (sequence, KV head): the CTAs cut the
// signature row into equal contiguous slices.
//   pass 1  every CTA streams its slice (16-byte loads, the next tile requested before the current one is counted)
//           into a histogram in shared memory (one counter per level and lane);
//   merge   the CTA histograms meet through distributed shared memory: every CTA reads all of them and derives the
//           same threshold T (largest level with #{S >= T} >= k), r = k - #{S > T}, and how many tokens with
//           S > T / S == T lie before its slice;
//   pass 2  takes the scores of pass 1 from shared memory (one byte per token, groups of up to four heads, slices of up
//           to 16384 / 65536 tokens; a one-tile slice keeps them in registers; anything else is scored again from L2)
//           and the selected tokens are written at their final positions: position = #{selected tokens
//           with a smaller index}, from a prefix sum over lanes, loads and warps.
// Nothing is kept in global scratch.  Tokens that are always in context (first n_sink, most recent n_local) are
// written without being scored, exactly as in the maximum variant.
// With groups of one head (G = 1, where sum, maximum and Eq. 1 coincide) and one unit per QUERY head the same kernel
// gives every query head its own list on the signature row of its KV head (row_shift).
#include "ha_score_dev.cuh"

namespace ha {

constexpr int kSumThreads = 256;
constexpr int kSumWarps = kSumThreads / 32;
// A tile is LD 16-byte loads per lane: 128 LD tokens per warp, 1024 LD per CTA (LD = 4 where few CTAs run and each
// must keep many bytes in flight, 2 where many CTAs share an SM and registers decide how many fit).
constexpr int kSumForced = -2, kSumAbsent = -1;                 // score stand-ins: always in context / outside the slice

struct SumArgs {
    const uint32_t *q_codes, *k_codes;
    long long kc_sb, kc_sh;
    const int32_t *seq_lens, *k_per_seq;
    int k_uniform, k_max, Hq, Hkv;
    int32_t *idx;
    long long idx_sb, idx_sh;
    int32_t *count, *hist_out;
    Windows win;
    int cache_tokens;   // score bytes that fit in the dynamic shared memory of one CTA
    int row_shift;      // unit head h scans the signature row of KV head h >> row_shift (per-query-head lists)
};

// The summed score without one population count per head: for bit position i let c_i = number of the group's query
// signatures with bit i set, d_i = G - c_i.  A key with bit i set agrees with c_i heads there, otherwise with d_i, so
// S = sum_i (k_i ? c_i : d_i) = sum_p 2^p popc((k & C_p) | (~k & D_p)) with C_p / D_p the bit planes of c / d:
// log2(G) + 1 population counts per token instead of G.
template <int G>
struct SumPlanes {
    static constexpr int P = (G == 1) ? 1 : (G == 2) ? 2 : (G == 4) ? 3 : 4;
    uint32_t C[P], D[P];
    __device__ __forceinline__ void build(const uint32_t (&q)[G]) {
#pragma unroll
        for (int p = 0; p < P; ++p) { C[p] = 0u; D[p] = 0u; }
#pragma unroll
        for (int j = 0; j < G; ++j) {   // bit-sliced counters: add the one-bit numbers q_j (and their complements)
            uint32_t carry_c = q[j], carry_d = ~q[j];
#pragma unroll
            for (int p = 0; p < P; ++p) {
                const uint32_t tc = C[p] & carry_c, td = D[p] & carry_d;
                C[p] ^= carry_c; D[p] ^= carry_d;
                carry_c = tc; carry_d = td;
            }
        }
    }
    __device__ __forceinline__ int score(uint32_t k) const {
        int s = 0;
#pragma unroll
        for (int p = 0; p < P; ++p) s += __popc((k & C[p]) | (~k & D[p])) << p;
        return s;
    }
};

// Scores of the 4 LD tokens this lane owns in a warp tile starting at `base`: load j covers tokens
// base + j * 128 + 4 * lane .. + 3.  kEdge: the tile may touch the always-kept windows or the end of the slice.
template <int G, int LD, bool kEdge>
__device__ __forceinline__ void sum_scores_of(const uint4 (&v)[LD], int base, int lane, int hi, WindowBounds wb,
                                              const SumPlanes<G> &pl, int (&sc)[4 * LD]) {
#pragma unroll
    for (int j = 0; j < LD; ++j) {
        const uint32_t c[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int s = pl.score(c[e]);
            if (kEdge) {
                const int t = base + j * 128 + 4 * lane + e;
                if (t < wb.sink_end || t >= wb.local_begin) s = kSumForced;
                if (t >= hi) s = kSumAbsent;
            }
            sc[4 * j + e] = s;
        }
    }
}

template <int LD, bool kEdge>
__device__ __forceinline__ void sum_load_tile(const uint32_t *row, int base, int lane, int hi, uint4 (&v)[LD]) {
#pragma unroll
    for (int j = 0; j < LD; ++j) {
        const int t = base + j * 128 + 4 * lane;
        if (kEdge) v[j] = (t < hi) ? load_codes4(row, t, hi) : make_uint4(0u, 0u, 0u, 0u);
        else v[j] = __ldg(reinterpret_cast<const uint4 *>(row + t));
    }
}

template <int G, int CS, int LD>
__global__ void __launch_bounds__(kSumThreads, LD <= 2 ? 5 : 3) score_sum_select_kernel(const SumArgs a) {
    constexpr int kWarpTokens = 128 * LD, kTileTokens = kSumWarps * kWarpTokens;
    constexpr int NB = 32 * G + 1;                      // score levels
    constexpr int kPer = (NB + 31) / 32;                // levels per lane in the threshold search
    __shared__ __align__(16) int c_hist[NB][32];        // pass 1: one counter per (level, lane): no two lanes of a warp meet
    __shared__ int s_hist[NB];                          // this CTA's histogram, read by the whole cluster
    __shared__ int s_tot[NB], s_bef[NB];                // whole sequence / slices before this one
    __shared__ int s_wsum[2][kSumWarps];                // pass 2: packed (S > T, S == T) counts per warp, double buffered
    __shared__ int s_T, s_r, s_gtb, s_eqb;
    // Scores of pass 1, one byte per token (levels 0 .. 128: groups of up to four heads), for slices that fit: pass 2
    // then neither reloads nor scores again, and compares four tokens per instruction.
    extern __shared__ uint32_t s_sc[];
    constexpr bool kCache = (G <= 4);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = (CS > 1) ? cluster_rank() : 0u;
    const int g = blockIdx.y, b = blockIdx.z;
    const int n = max(a.seq_lens[b], 0);
    const WindowBounds wb = window_bounds(a.win, n);
    const int nf = forced_before(wb, n);
    const int kb = a.k_per_seq ? a.k_per_seq[b] : a.k_uniform;
    const int keep = max(0, min(min(kb, a.k_max - nf), n - nf));     // heavy tokens retrieved among the others
    const uint32_t *row = a.k_codes + (long long)b * a.kc_sb + (long long)(g >> a.row_shift) * a.kc_sh;
    int32_t *list = a.idx + (long long)b * a.idx_sb + (long long)g * a.idx_sh;

    SumPlanes<G> pl;
    {
        uint32_t q[G];
#pragma unroll
        for (int j = 0; j < G; ++j) q[j] = __ldg(a.q_codes + (long long)b * a.Hq + (long long)g * G + j);
        pl.build(q);
    }

    // slice of this CTA: a multiple of four tokens, so that every 16-byte load stays inside it
    const int per = ((n + 3) / 4 + CS - 1) / CS * 4;
    const int lo = min(n, (int)rank * per), hi = min(n, lo + per);
    const int n_tiles = (hi - lo + kTileTokens - 1) / kTileTokens;
    const bool cached = kCache && n_tiles > 1 && hi - lo <= a.cache_tokens;   // a one-tile slice keeps its scores in registers
    const int plain_end = min(wb.local_begin, hi);      // warp tiles inside [sink_end, plain_end) need no per-token checks
    auto is_edge = [&](int base) { return base < wb.sink_end || base + kWarpTokens > plain_end; };

    for (int i = tid; i < NB * 8; i += kSumThreads) reinterpret_cast<uint4 *>(&c_hist[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();

    // ---- pass 1: histogram of the slice
    int sc[4 * LD];
    {
        uint4 v[LD], nx[LD];
        auto load = [&](int base, uint4 (&dst)[LD]) {
            if (is_edge(base)) sum_load_tile<LD, true>(row, base, lane, hi, dst);
            else sum_load_tile<LD, false>(row, base, lane, hi, dst);
        };
        if (n_tiles > 0) load(lo + warp * kWarpTokens, v);
        for (int it = 0; it < n_tiles; ++it) {
            const int base = lo + it * kTileTokens + warp * kWarpTokens;
            if (it + 1 < n_tiles) load(base + kTileTokens, nx);
            if (is_edge(base)) {
                sum_scores_of<G, LD, true>(v, base, lane, hi, wb, pl, sc);
#pragma unroll
                for (int e = 0; e < 4 * LD; ++e)
                    if (sc[e] >= 0) atomicAdd(&c_hist[sc[e]][lane], 1);
            } else {
                sum_scores_of<G, LD, false>(v, base, lane, hi, wb, pl, sc);
#pragma unroll
                for (int e = 0; e < 4 * LD; ++e) atomicAdd(&c_hist[sc[e]][lane], 1);
                if (cached) {
#pragma unroll
                    for (int j = 0; j < LD; ++j)
                        s_sc[(base - lo) / 4 + j * 32 + lane] = (uint32_t)sc[4 * j] | ((uint32_t)sc[4 * j + 1] << 8) |
                                                                 ((uint32_t)sc[4 * j + 2] << 16) | ((uint32_t)sc[4 * j + 3] << 24);
                }
            }
            if (it + 1 < n_tiles) {
#pragma unroll
                for (int j = 0; j < LD; ++j) v[j] = nx[j];
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < (NB + 31) / 32 * 32 * 8; i += kSumThreads) {   // eight threads per level, four counters each
        const int l = i >> 3;
        int s = 0;
        if (l < NB) {
            const uint4 c4 = reinterpret_cast<const uint4 *>(&c_hist[l][0])[i & 7];
            s = (int)(c4.x + c4.y + c4.z + c4.w);
        }
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        s += __shfl_xor_sync(0xffffffffu, s, 4);
        if (l < NB && (i & 7) == 0) { s_hist[l] = s; if (CS == 1) { s_tot[l] = s; s_bef[l] = 0; } }
    }
    if (CS > 1) {
        cluster_sync_all();   // every CTA's histogram is complete and visible
        // ---- merge: totals over the cluster and over the slices before this one (all remote loads issued, then added)
        for (int l = tid; l < NB; l += kSumThreads) {
            int x[CS];
#pragma unroll
            for (int r = 0; r < CS; ++r) x[r] = ld_dsmem(&s_hist[l], (uint32_t)r);
            int tot = 0, bef = 0;
#pragma unroll
            for (int r = 0; r < CS; ++r) { tot += x[r]; if (r < (int)rank) bef += x[r]; }
            s_tot[l] = tot;
            s_bef[l] = bef;
        }
        cluster_arrive();     // done reading the others' shared memory; matched by the wait at the end
    }
    __syncthreads();

    if (warp == 0) {      // threshold: lane l looks at levels [l * kPer, l * kPer + kPer)
        const int l0 = lane * kPer, l1 = min(NB, l0 + kPer);
        int mine = 0;
        for (int l = l0; l < l1; ++l) mine += s_tot[l];
        int suf = mine;   // tokens at the levels of lanes >= this one
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
            const int o = __shfl_down_sync(0xffffffffu, suf, dd);
            if (lane + dd < 32) suf += o;
        }
        int above = suf - mine, T = NB, r = 0;
        bool found = false;
        if (keep > 0) {
            for (int l = l1 - 1; l >= l0; --l) {
                const int here = s_tot[l];
                if (!found && above < keep && keep <= above + here) { found = true; T = l; r = keep - above; }
                above += here;
            }
        }
        const unsigned who = __ballot_sync(0xffffffffu, found);
        const int src = who ? (__ffs(who) - 1) : 0;
        T = __shfl_sync(0xffffffffu, T, src);
        r = __shfl_sync(0xffffffffu, r, src);
        int gtb = 0;
        for (int l = l0; l < l1; ++l)
            if (l > T) gtb += s_bef[l];
#pragma unroll
        for (int dd = 16; dd > 0; dd >>= 1) gtb += __shfl_xor_sync(0xffffffffu, gtb, dd);
        if (lane == 0) { s_T = T; s_r = r; s_gtb = gtb; s_eqb = (T < NB) ? s_bef[T] : 0; }
    }
    __syncthreads();
    const int T = s_T, r = s_r;
    if (a.hist_out && rank == 0)
        for (int l = tid; l < NB; l += kSumThreads) a.hist_out[((long long)b * a.Hkv + g) * NB + l] = s_tot[l];

    // ---- pass 2: the selected tokens of the slice, at their final positions
    const int local_pos0 = wb.sink_end + keep;   // where the most recent tokens go
    int run_g = s_gtb, run_q = s_eqb;            // tokens with S > T / S == T before the current tile
    for (int it = 0; it < n_tiles; ++it) {
        const int base = lo + it * kTileTokens + warp * kWarpTokens;
        const bool edge = is_edge(base);
        // bit i of the masks: token i of this lane (load i / 4, element i % 4) has S > T / S == T / is always kept
        uint32_t gtm = 0, eqm = 0, fm = 0;
        if (cached && !edge) {   // score bytes of pass 1, four tokens per comparison (T <= 129 fits a byte)
            const uint32_t t4 = (uint32_t)T * 0x01010101u;
#pragma unroll
            for (int j = 0; j < LD; ++j) {
                const uint32_t w = s_sc[(base - lo) / 4 + j * 32 + lane];
                gtm |= high_bits_to_nibble(__vcmpgtu4(w, t4)) << (4 * j);
                eqm |= high_bits_to_nibble(__vcmpeq4(w, t4)) << (4 * j);
            }
        } else {
            if (n_tiles != 1) {   // a slice of one tile still holds its scores in registers
                uint4 v[LD];
                if (edge) { sum_load_tile<LD, true>(row, base, lane, hi, v); sum_scores_of<G, LD, true>(v, base, lane, hi, wb, pl, sc); }
                else { sum_load_tile<LD, false>(row, base, lane, hi, v); sum_scores_of<G, LD, false>(v, base, lane, hi, wb, pl, sc); }
            }
#pragma unroll
            for (int i = 0; i < 4 * LD; ++i) {
                gtm |= (sc[i] > T ? 1u : 0u) << i;
                eqm |= (sc[i] == T ? 1u : 0u) << i;
                if (edge) fm |= (sc[i] == kSumForced ? 1u : 0u) << i;
            }
        }
        // packed counts (S > T in the low half, S == T in the high half) of this lane per load, then over the warp
        int excl[LD], warp_total = 0;
#pragma unroll
        for (int j = 0; j < LD; ++j) {
            // bits set in the two nibbles, on the integer pipe (the population-count unit is the busy one here)
            uint32_t v = ((gtm >> (4 * j)) & 15u) | (((eqm >> (4 * j)) & 15u) << 16);
            v -= (v >> 1) & 0x00050005u;
            const int p = (int)((v & 0x00030003u) + ((v >> 2) & 0x00030003u));
            int inc = p;
#pragma unroll
            for (int dd = 1; dd < 32; dd <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, inc, dd);
                if (lane >= dd) inc += o;
            }
            excl[j] = warp_total + inc - p;
            warp_total += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) s_wsum[it & 1][warp] = warp_total;
        __syncthreads();
        int before = 0, tile_total = 0;
#pragma unroll
        for (int w = 0; w < kSumWarps; ++w) {
            const int x = s_wsum[it & 1][w];
            if (w < warp) before += x;
            tile_total += x;
        }
        // A token with S > T, or one of the first r with S == T, lands behind everything selected before it:
        // #{S > T before} + min(#{S == T before}, r).
        if (LD >= 4) {
            // few CTAs, each alone on its SM: only the few tokens at or above the threshold are visited
            for (uint32_t m = gtm | eqm; m; m &= m - 1) {
                const int i = __ffs(m) - 1, j = i >> 2, e = i & 3;
                int ex = excl[0];
#pragma unroll
                for (int jj = 1; jj < LD; ++jj)
                    if (j == jj) ex = excl[jj];
                const uint32_t low = (1u << e) - 1u;
                const int gb = run_g + ((before + ex) & 0xffff) + __popc((gtm >> (4 * j)) & low);
                const int qb = run_q + ((before + ex) >> 16) + __popc((eqm >> (4 * j)) & low);
                if (((gtm >> i) & 1u) || qb < r) list[wb.sink_end + gb + min(qb, r)] = base + j * 128 + 4 * lane + e;
            }
        } else {
            // many CTAs per SM, bound by instruction issue: straight-line code, one predicated store per token
#pragma unroll
            for (int j = 0; j < LD; ++j) {
                int gb = run_g + ((before + excl[j]) & 0xffff), qb = run_q + ((before + excl[j]) >> 16);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool gt = (gtm >> (4 * j + e)) & 1u, eq = (eqm >> (4 * j + e)) & 1u;
                    if (gt || (eq && qb < r)) list[wb.sink_end + gb + min(qb, r)] = base + j * 128 + 4 * lane + e;
                    gb += gt ? 1 : 0;
                    qb += eq ? 1 : 0;
                }
            }
        }
        for (uint32_t m = fm; m; m &= m - 1) {   // edge tiles only
            const int i = __ffs(m) - 1, t = base + (i >> 2) * 128 + 4 * lane + (i & 3);
            list[t < wb.sink_end ? t : local_pos0 + (t - wb.local_begin)] = t;
        }
        run_g += tile_total & 0xffff;
        run_q += tile_total >> 16;
    }

    // ---- count and padding
    const int cnt = nf + keep;
    if (rank == 0 && tid == 0) a.count[(long long)b * a.Hkv + g] = cnt;
    for (int i = cnt + (int)rank * kSumThreads + tid; i < a.k_max; i += CS * kSumThreads) list[i] = -1;
    if (CS > 1) cluster_wait();
}

template <int G, int CS, int LD>
static cudaError_t launch_sum_t(const SumArgs &a, int B, cudaStream_t st) {
    if (CS > 8) {   // clusters of more than 8 CTAs are an opt-in, per device
        static bool allowed[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev < 0 || dev >= 64) dev = 0;
        if (!allowed[dev]) {
            cudaError_t e = cudaFuncSetAttribute(score_sum_select_kernel<G, CS, LD>,
                                                 cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e != cudaSuccess) return e;
            allowed[dev] = true;
        }
    }
    // score bytes of pass 1 (groups of up to four heads): 16 KB where five CTAs share an SM; 64 KB in the few-CTA variant,
    // which still lets two CTAs share an SM (with one per SM only seven clusters of 16 are resident at a time)
    constexpr int kCacheBytes = (G > 4) ? 0 : (LD >= 4 ? 64 * 1024 : 16 * 1024);
    if (kCacheBytes > 24 * 1024) {
        static bool sized[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev < 0 || dev >= 64) dev = 0;
        if (!sized[dev]) {
            cudaError_t e = cudaFuncSetAttribute(score_sum_select_kernel<G, CS, LD>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, kCacheBytes);
            if (e != cudaSuccess) return e;
            sized[dev] = true;
        }
    }
    SumArgs args = a;
    args.cache_tokens = kCacheBytes;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS, a.Hkv, B);
    cfg.blockDim = dim3(kSumThreads);
    cfg.dynamicSmemBytes = kCacheBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, score_sum_select_kernel<G, CS, LD>, args);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

// CTAs per unit: enough to give every SM about four CTAs, in clusters of at most 8 (16 for a handful of units, whose
// sequences may be long).  The sequence lengths live on the device, so the choice looks at the unit count only;
// a CTA whose slice is empty only takes part in the exchange.
template <int G>
static cudaError_t launch_sum_g(const SumArgs &a, int B, cudaStream_t st) {
    const long long units = (long long)B * a.Hkv, want = 4LL * sm_count();
    if (units * 8 < sm_count()) return launch_sum_t<G, 16, 4>(a, B, st);
    if (units * 4 < want) return launch_sum_t<G, 8, 2>(a, B, st);
    if (units * 2 < want) return launch_sum_t<G, 4, 2>(a, B, st);
    if (units < want) return launch_sum_t<G, 2, 2>(a, B, st);
    return launch_sum_t<G, 1, 2>(a, B, st);
}

cudaError_t launch_score_topk_sum(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes, long long kc_sb,
                                  long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq, int k_uniform,
                                  int k_max, int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                                  int32_t *hist_out, cudaStream_t st, Windows win, bool per_head) {
    if (B <= 0 || Hkv <= 0) return cudaSuccess;
    SumArgs a;
    a.q_codes = q_codes; a.k_codes = k_codes; a.kc_sb = kc_sb; a.kc_sh = kc_sh;
    a.seq_lens = seq_lens; a.k_per_seq = k_per_seq; a.k_uniform = k_uniform; a.k_max = k_max;
    a.Hq = Hq; a.Hkv = Hkv; a.idx = idx; a.idx_sb = idx_sb; a.idx_sh = idx_sh;
    a.count = count; a.hist_out = hist_out; a.win = win; a.cache_tokens = 0; a.row_shift = 0;
    if (per_head) {   // every query head is a unit of its own (one head per group) on the row of its KV head
        int shift = 0;
        while ((Hkv << shift) < Hq) ++shift;
        a.Hkv = Hq;
        a.row_shift = shift;
        return launch_sum_g<1>(a, B, st);
    }
    switch (Hq / Hkv) {
        case 1: return launch_sum_g<1>(a, B, st);
        case 2: return launch_sum_g<2>(a, B, st);
        case 4: return launch_sum_g<4>(a, B, st);
        case 8: return launch_sum_g<8>(a, B, st);
        default: return cudaErrorInvalidValue;
    }
}

} // namespace ha
