// SCORE + TOPK for signatures of b = 64 .. 512 bits kept as b/64 packed 64-bit integers (the widths of the paper's
// bit-width study and of its table "Latency of SCORE computation"): Eq. 1 with the bitcount(xor) identity of Section
// 4.1 at b bits, s = b - popcount(k xor q), reduced with max over the query heads of a GQA group as in the 32-bit
// layer-step, then the standard top-k of Section 4 with ties towards the lowest token index.  Scores take b + 1
// values, so the selection is again a histogram threshold plus an index-ordered compaction, never a sort.
//
// Three kernels over chunks of every (sequence, KV head) unit, each at full parallelism, nothing waits:
//   1. wide_scan_kernel      streams the signatures, leaves one 16-bit score per token in the workspace and adds the
//                            chunk's level counts to the unit's (b + 1)-level histogram;
//   2. wide_count_kernel     every chunk derives the threshold T (largest level with #{S >= T} >= k) from the unit's
//                            histogram and counts its own tokens above / at T;
//   3. wide_write_kernel     every chunk adds up the counts of the chunks before it and writes its selected tokens at
//                            their final positions (ascending token index; the first r = k - #{S > T} tokens at T).
// Tokens that are always in context (the first n_sink, the most recent n_local) carry the score 0xFFFF, which is
// above every threshold, and are left out of the histogram.
#include "ha_score_dev.cuh"

namespace ha {

constexpr int kWideThreads = 256;
constexpr int kWideMaxLevels = 513;            // scores 0 .. 512
constexpr int kWideHistStride = 520;
constexpr int kWideTokensPerThread = 16;
constexpr int kWidePass = kWideThreads * kWideTokensPerThread;   // tokens of one pass of a CTA
constexpr uint32_t kWideForced = 0xFFFFu;
constexpr int kWideMaxChunks = 1024;           // chunks per unit: a single long sequence still fills the device

struct WideArgs {
    const uint64_t *q_codes, *k_codes;
    long long kc_sb, kc_sh;        // in 64-bit words
    const int32_t *seq_lens, *k_per_seq;
    int k_uniform, max_seq_len, k_max, Hq, Hkv, G, n_bits, chunk_tokens;
    Windows win;
    int32_t *idx;
    long long idx_sb, idx_sh;
    int32_t *count, *hist_out;
    int32_t *unit_hist;            // [units][kWideHistStride], zero before the scan
    int32_t *chunk_counts;         // [units][kWideMaxChunks][2]
    uint16_t *scores;              // [units][score_row]
    long long score_row;
};

struct WideUnit {
    int n, keep, keep_rest;
    WindowBounds wbd;
};
__device__ __forceinline__ WideUnit wide_unit(const WideArgs &a, int b) {
    WideUnit r;
    r.n = max(min(a.seq_lens[b], a.max_seq_len), 0);
    const int k = a.k_per_seq ? a.k_per_seq[b] : a.k_uniform;
    r.wbd = window_bounds(a.win, r.n);
    const int nf = forced_before(r.wbd, r.n);
    r.keep_rest = max(0, min(min(k, a.k_max - nf), r.n - nf));
    r.keep = nf + r.keep_rest;
    return r;
}

template <int W>
__global__ void __launch_bounds__(kWideThreads) wide_scan_kernel(const WideArgs a) {
    __shared__ int s_hist[kWideThreads / 32][kWideMaxLevels + 7];   // one table per warp
    __shared__ unsigned long long s_q[kMaxGroup][W];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5;
    const WideUnit wu = wide_unit(a, b);
    const int start = chunk * a.chunk_tokens;
    if (start >= wu.n) return;
    const int end = min(wu.n, start + a.chunk_tokens);
    const int levels = a.n_bits + 1;
    for (int i = tid; i < (kWideThreads / 32) * (kWideMaxLevels + 7); i += kWideThreads) (&s_hist[0][0])[i] = 0;
    if (tid < a.G * W) s_q[tid / W][tid % W] = a.q_codes[((long long)b * a.Hq + (long long)g * a.G + tid / W) * W + tid % W];
    __syncthreads();
    const int unit = b * a.Hkv + g;
    const uint64_t *row = a.k_codes + (long long)b * a.kc_sb + (long long)g * a.kc_sh;
    uint16_t *srow = a.scores + (long long)unit * a.score_row;
    for (int t = start + tid; t < end; t += kWideThreads) {   // a warp reads 32 W consecutive words per step
        unsigned long long kw[W];
        if (W == 1) {
            kw[0] = __ldg(reinterpret_cast<const unsigned long long *>(row + t));
        } else {
#pragma unroll
            for (int w = 0; w < W; w += 2) {
                const ulonglong2 v = __ldg(reinterpret_cast<const ulonglong2 *>(row + (long long)t * W + w));
                kw[w] = v.x; kw[w + 1] = v.y;
            }
        }
        int best = a.n_bits + 1;   // smallest Hamming distance over the group
        for (int j = 0; j < a.G; ++j) {
            int h = 0;
#pragma unroll
            for (int w = 0; w < W; ++w) h += __popcll(kw[w] ^ s_q[j][w]);
            best = min(best, h);
        }
        const int score = a.n_bits - best;
        const bool forced = t < wu.wbd.sink_end || t >= wu.wbd.local_begin;
        srow[t] = forced ? (uint16_t)kWideForced : (uint16_t)score;
        // unrelated signatures crowd into a few levels around b / 2: lanes with the same score add once, together
        const int key = forced ? -1 : score;
        const unsigned peers = __match_any_sync(__activemask(), key);
        if (key >= 0 && (int)(__ffs(peers) - 1) == (tid & 31)) atomicAdd(&s_hist[warp][score], __popc(peers));
    }
    __syncthreads();
    int32_t *uh = a.unit_hist + (long long)unit * kWideHistStride;
    for (int l = tid; l < levels; l += kWideThreads) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < kWideThreads / 32; ++w) c += s_hist[w][l];
        if (c) atomicAdd(uh + l, c);
    }
}

// Threshold of a unit from its level counts in shared memory (levels = b + 1), by warp 0: T = largest level with
// #{S >= T} >= keep (levels if keep == 0: nothing is selected by score), gt = #{S > T}.  Result in every lane.
__device__ __forceinline__ void wide_threshold(const int *hist, int levels, int keep, int lane, int &T, int &gt) {
    const int per = (levels + 31) / 32;
    const int lo = min(levels, lane * per), hi = min(levels, lo + per);
    int seg = 0;
    for (int l = lo; l < hi; ++l) seg += hist[l];
    int above = seg;   // inclusive suffix sum over lanes: levels >= lo
#pragma unroll
    for (int dd = 1; dd < 32; dd <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, above, dd);
        if (lane + dd < 32) above += v;
    }
    T = levels; gt = 0;
    if (keep <= 0) return;
    const unsigned ok = __ballot_sync(0xffffffffu, above >= keep);   // lanes whose lowest level already has enough above it
    if (ok == 0u) { T = 0; gt = __shfl_sync(0xffffffffu, above, 0) - hist[0]; return; }   // cannot happen: #{S >= 0} = n >= keep
    const int owner = 31 - __clz(ok);
    int myT = 0, mygt = 0;
    if (lane == owner) {
        int c = above - seg;   // levels above this lane's segment
        for (int l = hi - 1; l >= lo; --l) {
            if (c + hist[l] >= keep) { myT = l; mygt = c; break; }
            c += hist[l];
        }
    }
    T = __shfl_sync(0xffffffffu, myT, owner);
    gt = __shfl_sync(0xffffffffu, mygt, owner);
}

// flags of 16 consecutive tokens from `first` on (bit i = token first + i): score > T (always-kept tokens included) / == T
__device__ __forceinline__ void wide_flags16(const uint16_t *srow, int first, int end, int T, uint32_t &gt, uint32_t &eq) {
    gt = 0u; eq = 0u;
    if (first >= end) return;
    const uint4 v0 = __ldcg(reinterpret_cast<const uint4 *>(srow + first)), v1 = __ldcg(reinterpret_cast<const uint4 *>(srow + first + 8));
    const uint32_t wv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const int s = (int)((wv[e >> 1] >> (16 * (e & 1))) & 0xffffu);
        if (first + e < end) {
            gt |= (uint32_t)(s > T) << e;
            eq |= (uint32_t)(s == T) << e;
        }
    }
}

__global__ void __launch_bounds__(kWideThreads) wide_count_kernel(const WideArgs a) {
    __shared__ int s_hist[kWideMaxLevels + 7];
    __shared__ int s_T, s_red[2][kWideThreads / 32];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const WideUnit wu = wide_unit(a, b);
    const int start = chunk * a.chunk_tokens;
    if (start >= wu.n && chunk > 0) return;
    const int end = min(wu.n, start + a.chunk_tokens);
    const int unit = b * a.Hkv + g, levels = a.n_bits + 1;
    const int32_t *uh = a.unit_hist + (long long)unit * kWideHistStride;
    for (int l = tid; l < levels; l += kWideThreads) s_hist[l] = __ldcg(uh + l);
    __syncthreads();
    if (warp == 0) {
        int T, gt;
        wide_threshold(s_hist, levels, wu.keep_rest, lane, T, gt);
        if (lane == 0) s_T = T;
    }
    __syncthreads();
    const int T = s_T;
    const uint16_t *srow = a.scores + (long long)unit * a.score_row;
    int cg = 0, ce = 0;
    for (int first = start + tid * kWideTokensPerThread; first < end; first += kWidePass) {
        uint32_t gt, eq;
        wide_flags16(srow, first, end, T, gt, eq);
        cg += __popc(gt); ce += __popc(eq);
    }
#pragma unroll
    for (int dd = 16; dd > 0; dd >>= 1) { cg += __shfl_xor_sync(0xffffffffu, cg, dd); ce += __shfl_xor_sync(0xffffffffu, ce, dd); }
    if (lane == 0) { s_red[0][warp] = cg; s_red[1][warp] = ce; }
    __syncthreads();
    if (tid < 2) {
        int s = 0;
        for (int w = 0; w < kWideThreads / 32; ++w) s += s_red[tid][w];
        a.chunk_counts[((long long)unit * kWideMaxChunks + chunk) * 2 + tid] = s;
    }
}

__global__ void __launch_bounds__(kWideThreads) wide_write_kernel(const WideArgs a) {
    __shared__ int s_hist[kWideMaxLevels + 7];
    __shared__ int s_T, s_gt, s_before[2], s_wtot[kWideThreads / 32];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const WideUnit wu = wide_unit(a, b);
    const int start = chunk * a.chunk_tokens;
    if (start >= wu.n && chunk > 0) return;
    const int end = min(wu.n, start + a.chunk_tokens);
    const int unit = b * a.Hkv + g, levels = a.n_bits + 1;
    const int32_t *uh = a.unit_hist + (long long)unit * kWideHistStride;
    for (int l = tid; l < levels; l += kWideThreads) s_hist[l] = __ldcg(uh + l);
    if (tid < 2) s_before[tid] = 0;
    __syncthreads();
    if (warp == 0) {
        int T, gt;
        wide_threshold(s_hist, levels, wu.keep_rest, lane, T, gt);
        if (lane == 0) { s_T = T; s_gt = gt; }
    } else if (warp <= 2) {   // tokens above / at the threshold in the chunks before this one
        const int which = warp - 1;
        int s = 0;
        for (int c = lane; c < chunk; c += 32) s += __ldcg(a.chunk_counts + ((long long)unit * kWideMaxChunks + c) * 2 + which);
#pragma unroll
        for (int dd = 16; dd > 0; dd >>= 1) s += __shfl_xor_sync(0xffffffffu, s, dd);
        if (lane == 0) s_before[which] = s;
    }
    __syncthreads();
    const int T = s_T, r = wu.keep_rest - s_gt;   // tokens of score exactly T that are still wanted
    int32_t *list = a.idx + (long long)b * a.idx_sb + (long long)g * a.idx_sh;
    if (chunk == 0) {
        if (tid == 0) a.count[unit] = wu.keep;
        for (int i = wu.keep + tid; i < a.k_max; i += kWideThreads) list[i] = -1;
        if (a.hist_out) for (int l = tid; l < levels; l += kWideThreads) a.hist_out[(long long)unit * levels + l] = s_hist[l];
    }
    if (wu.keep == 0) return;
    const uint16_t *srow = a.scores + (long long)unit * a.score_row;
    int run_gt = s_before[0], run_eq = s_before[1];
    for (int pass = start; pass < end; pass += kWidePass) {   // CTA-uniform
        const int first = pass + tid * kWideTokensPerThread;
        uint32_t gt, eq;
        wide_flags16(srow, first, end, T, gt, eq);
        const int packed = __popc(gt) | (__popc(eq) << 16);
        int inc = packed;
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, dd);
            if (lane >= dd) inc += v;
        }
        if (lane == 31) s_wtot[warp] = inc;
        __syncthreads();
        int wpre = 0, all = 0;
#pragma unroll
        for (int w = 0; w < kWideThreads / 32; ++w) {
            const int v = s_wtot[w];
            if (w < warp) wpre += v;
            all += v;
        }
        if (packed != 0) {
            const int excl = wpre + inc - packed;
            int g_run = run_gt + (excl & 0xffff), q_run = run_eq + (int)((unsigned)excl >> 16);
            write_selected32(list, first, gt, eq, g_run, q_run, r);
        }
        run_gt += all & 0xffff;
        run_eq += (int)((unsigned)all >> 16);
        __syncthreads();
    }
}

// Workspace of the wide selection: header | unit histograms | chunk counts | 16-bit scores.
struct WideLayout {
    size_t off_hist, off_counts, off_scores, score_row, total;
};
WideLayout wide_layout(int B, int Hkv, int max_seq_len) {
    WideLayout L;
    const size_t units = (size_t)B * Hkv;
    size_t o = kHeaderBytes;
    L.off_hist = o;   o = align_up(o + units * kWideHistStride * 4, 256);
    L.off_counts = o; o = align_up(o + units * kWideMaxChunks * 2 * 4, 256);
    L.score_row = align_up((size_t)(max_seq_len > 0 ? max_seq_len : 0), 256);
    L.off_scores = o; o = align_up(o + units * L.score_row * 2, 256);
    L.total = o;
    return L;
}
size_t wide_workspace_bytes(int B, int Hkv, int max_seq_len) { return wide_layout(B, Hkv, max_seq_len).total; }

cudaError_t launch_score_topk_wide(int B, int Hq, int Hkv, int n_bits, const uint64_t *q_codes, const uint64_t *k_codes,
                                   long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq,
                                   int k_uniform, int max_seq_len, int k_max, int32_t *idx, long long idx_sb, long long idx_sh,
                                   int32_t *count, int32_t *hist_out, void *workspace, cudaStream_t st, Windows win) {
    const WideLayout L = wide_layout(B, Hkv, max_seq_len);
    char *ws = reinterpret_cast<char *>(workspace);
    WideArgs a{};
    a.q_codes = q_codes; a.k_codes = k_codes; a.kc_sb = kc_sb; a.kc_sh = kc_sh; a.seq_lens = seq_lens; a.k_per_seq = k_per_seq;
    a.k_uniform = k_uniform; a.max_seq_len = max_seq_len; a.k_max = k_max; a.Hq = Hq; a.Hkv = Hkv; a.G = Hq / Hkv; a.n_bits = n_bits;
    a.win = win; a.idx = idx; a.idx_sb = idx_sb; a.idx_sh = idx_sh; a.count = count; a.hist_out = hist_out;
    a.unit_hist = reinterpret_cast<int32_t *>(ws + L.off_hist);
    a.chunk_counts = reinterpret_cast<int32_t *>(ws + L.off_counts);
    a.scores = reinterpret_cast<uint16_t *>(ws + L.off_scores);
    a.score_row = (long long)L.score_row;
    // chunks of whole passes, about eight CTAs per SM when there is that much work, at most kWideMaxChunks per unit
    const long long units = (long long)B * Hkv, n = max_seq_len > 0 ? max_seq_len : 1;
    long long per_unit = 8LL * sm_count() / (units > 0 ? units : 1);
    if (per_unit < 1) per_unit = 1;
    if (per_unit > kWideMaxChunks) per_unit = kWideMaxChunks;
    long long c = (n + per_unit - 1) / per_unit;
    const long long c_min = (n + kWideMaxChunks - 1) / kWideMaxChunks;
    if (c < c_min) c = c_min;
    if (c < kWidePass) c = kWidePass;
    a.chunk_tokens = (int)((c + kWidePass - 1) / kWidePass * kWidePass);
    const int n_chunks = (int)((n + a.chunk_tokens - 1) / a.chunk_tokens);
    cudaError_t e = cudaMemsetAsync(a.unit_hist, 0, (size_t)units * kWideHistStride * 4, st);
    if (e != cudaSuccess) return e;
    dim3 grid(n_chunks, Hkv, B);
    switch (n_bits / 64) {
        case 1: wide_scan_kernel<1><<<grid, kWideThreads, 0, st>>>(a); break;
        case 2: wide_scan_kernel<2><<<grid, kWideThreads, 0, st>>>(a); break;
        case 4: wide_scan_kernel<4><<<grid, kWideThreads, 0, st>>>(a); break;
        case 8: wide_scan_kernel<8><<<grid, kWideThreads, 0, st>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    wide_count_kernel<<<grid, kWideThreads, 0, st>>>(a);
    wide_write_kernel<<<grid, kWideThreads, 0, st>>>(a);
    count_launch(3);
    return cudaGetLastError();
}

} // namespace ha
