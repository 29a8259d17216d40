// SCORE + TOPK.  Scores are s = 32 - popc(k_code ^ q_code) (Eq. 1 via the bitcount-xor identity of
// Section 4.1), reduced with max over the query heads of the GQA group, so they take only 33
// values.  "Standard top-k" (Section 4) therefore needs no sort: a histogram gives the threshold
// score T and how many tokens r of score exactly T are still needed; the selection is every token
// above T plus the first r tokens at T in index order, written in ascending token order.
//
// Kernel 1 (scan_hist): each CTA streams one chunk of the code cache with 16-byte loads and
//   leaves the chunk's 33-bin histogram in the workspace.
// Kernel 2 (select): each CTA sums the chunk histograms (total, and the part before its own
//   chunk), derives T, r and its output offset, re-reads its chunk (an L2 hit) and compacts the
//   selected token indices with warp-shuffle prefix sums.  No CTA waits on another.
#include "ha_common.cuh"

namespace ha {

constexpr int kScanThreads = 256;
constexpr int kScanTokensPerPass = kScanThreads * 4;   // one uint4 per thread

template <int G>
__device__ __forceinline__ int group_score(uint32_t code, const uint32_t (&qc)[G]) {
    int h = __popc(code ^ qc[0]);
#pragma unroll
    for (int j = 1; j < G; ++j) h = min(h, __popc(code ^ qc[j]));
    return kBits - h;
}

__device__ __forceinline__ uint4 load_codes4(const uint32_t *row, int base, int n) {
    // tokens base..base+3 of a 16-byte aligned row; tokens >= n come back as don't-care zeros
    if (base + 3 < n) return __ldg(reinterpret_cast<const uint4 *>(row + base));
    uint4 v = make_uint4(0, 0, 0, 0);
    if (base + 0 < n) v.x = __ldg(row + base + 0);
    if (base + 1 < n) v.y = __ldg(row + base + 1);
    if (base + 2 < n) v.z = __ldg(row + base + 2);
    return v;
}

template <int G>
__global__ void __launch_bounds__(kScanThreads) scan_hist_kernel(const uint32_t *__restrict__ q_codes,
                                                                const uint32_t *__restrict__ k_codes,
                                                                long long kc_sb, long long kc_sh,
                                                                const int32_t *__restrict__ seq_lens,
                                                                int max_seq_len, int Hq, int Hkv,
                                                                int chunk_tokens,
                                                                int32_t *__restrict__ ws_hist) {
    // 4 sub-histograms per warp (by lane & 3) spread same-bin updates over several addresses
    __shared__ int hist[kScanThreads / 32][4][kBins + 3];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int n = min(seq_lens[b], max_seq_len);
    const int start = chunk * chunk_tokens;
    if (start >= n) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int i = tid; i < (kScanThreads / 32) * 4 * (kBins + 3); i += kScanThreads) (&hist[0][0][0])[i] = 0;
    uint32_t qc[G];
#pragma unroll
    for (int j = 0; j < G; ++j) qc[j] = __ldg(q_codes + (long long)b * Hq + g * G + j);
    __syncthreads();

    const uint32_t *row = k_codes + (long long)b * kc_sb + (long long)g * kc_sh;
    const int end = min(n, start + chunk_tokens);
    int *my = hist[warp][lane & 3];
    for (int base = start + tid * 4; base < end; base += kScanTokensPerPass) {
        const uint4 c = load_codes4(row, base, end);
        atomicAdd(&my[group_score<G>(c.x, qc)], 1);
        if (base + 1 < end) atomicAdd(&my[group_score<G>(c.y, qc)], 1);
        if (base + 2 < end) atomicAdd(&my[group_score<G>(c.z, qc)], 1);
        if (base + 3 < end) atomicAdd(&my[group_score<G>(c.w, qc)], 1);
    }
    __syncthreads();
    if (tid < kBins) {
        int s = 0;
#pragma unroll
        for (int w = 0; w < kScanThreads / 32; ++w)
#pragma unroll
            for (int r = 0; r < 4; ++r) s += hist[w][r][tid];
        ws_hist[(((long long)b * Hkv + g) * kMaxChunks + chunk) * kBins + tid] = s;
    }
}

template <int G>
__global__ void __launch_bounds__(kScanThreads) select_kernel(const uint32_t *__restrict__ q_codes,
                                                             const uint32_t *__restrict__ k_codes,
                                                             long long kc_sb, long long kc_sh,
                                                             const int32_t *__restrict__ seq_lens,
                                                             int max_seq_len,
                                                             const int32_t *__restrict__ k_per_seq, int k_uniform,
                                                             int k_max, int Hq, int Hkv, int chunk_tokens,
                                                             const int32_t *__restrict__ ws_hist,
                                                             int32_t *__restrict__ idx, long long idx_sb,
                                                             long long idx_sh, int32_t *__restrict__ count,
                                                             int32_t *__restrict__ hist_out) {
    __shared__ int tot[kBins], bef[kBins];
    __shared__ int sh_T, sh_r, sh_gt_before, sh_eq_before;
    __shared__ int warp_tot[kScanThreads / 32];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = max(min(seq_lens[b], max_seq_len), 0);
    int k = k_per_seq ? k_per_seq[b] : k_uniform;
    k = max(0, min(k, k_max));
    const int keep = min(k, n);
    const int n_chunks = (n + chunk_tokens - 1) / chunk_tokens;
    if (chunk > 0 && chunk >= n_chunks) return;

    // totals per score level, and the part contributed by the chunks before this one
    if (tid < kBins) {
        const int32_t *hb = ws_hist + ((long long)b * Hkv + g) * kMaxChunks * kBins + tid;
        int t = 0, be = 0;
        for (int c = 0; c < n_chunks; ++c) {
            const int v = hb[c * kBins];
            t += v;
            if (c < chunk) be += v;
        }
        tot[tid] = t;
        bef[tid] = be;
    }
    __syncthreads();
    if (tid == 0) {
        // T = largest level with #{S >= T} >= keep; r = keep - #{S > T}
        int T = kBins, r = 0, cum = 0;
        if (keep > 0) {
            for (int t = kBins - 1; t >= 0; --t) {
                if (cum + tot[t] >= keep) { T = t; r = keep - cum; break; }
                cum += tot[t];
            }
        }
        int gb = 0;
        for (int t = T + 1; t < kBins; ++t) gb += bef[t];
        sh_T = T; sh_r = r; sh_gt_before = gb; sh_eq_before = (T < kBins) ? bef[T] : 0;
    }
    __syncthreads();
    const int T = sh_T, r = sh_r;
    int32_t *out = idx + (long long)b * idx_sb + (long long)g * idx_sh;
    if (chunk == 0) {
        if (tid == 0) count[b * Hkv + g] = keep;
        if (hist_out && tid < kBins) hist_out[((long long)b * Hkv + g) * kBins + tid] = tot[tid];
        for (int i = keep + tid; i < k_max; i += kScanThreads) out[i] = -1;
    }
    if (chunk >= n_chunks || keep == 0) return;

    uint32_t qc[G];
#pragma unroll
    for (int j = 0; j < G; ++j) qc[j] = __ldg(q_codes + (long long)b * Hq + g * G + j);
    const uint32_t *row = k_codes + (long long)b * kc_sb + (long long)g * kc_sh;
    const int start = chunk * chunk_tokens, end = min(n, start + chunk_tokens);
    int run_gt = sh_gt_before, run_eq = sh_eq_before;   // tokens before this pass with S > T / S == T

    for (int pass = start; pass < end; pass += kScanTokensPerPass) {
        const int base = pass + tid * 4;
        int s[4] = {-1, -1, -1, -1};
        if (base < end) {
            const uint4 c = load_codes4(row, base, end);
            s[0] = group_score<G>(c.x, qc);
            if (base + 1 < end) s[1] = group_score<G>(c.y, qc);
            if (base + 2 < end) s[2] = group_score<G>(c.z, qc);
            if (base + 3 < end) s[3] = group_score<G>(c.w, qc);
        }
        int cg = 0, ce = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) { cg += (s[e] > T); ce += (s[e] == T); }
        // block-wide exclusive prefix of (cg, ce), packed as two 16-bit counters (pass <= 1024 tokens)
        const int packed = cg | (ce << 16);
        int inc = packed;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += v;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        int wpre = 0, all = 0;
#pragma unroll
        for (int w = 0; w < kScanThreads / 32; ++w) {
            const int v = warp_tot[w];
            if (w < warp) wpre += v;
            all += v;
        }
        const int excl = wpre + inc - packed;
        int gt_lt = run_gt + (excl & 0xffff);
        int eq_lt = run_eq + (excl >> 16);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (s[e] > T) {
                out[gt_lt + min(eq_lt, r)] = base + e;
                ++gt_lt;
            } else if (s[e] == T) {
                if (eq_lt < r) out[gt_lt + eq_lt] = base + e;
                ++eq_lt;
            }
        }
        run_gt += all & 0xffff;
        run_eq += all >> 16;
        __syncthreads();   // warp_tot is rewritten by the next pass
    }
}

template <int G>
static cudaError_t launch_g(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes,
                            long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq,
                            int k_uniform, int max_seq_len, int k_max, int32_t *idx, long long idx_sb,
                            long long idx_sh, int32_t *count, int32_t *hist_out, int32_t *ws_hist,
                            cudaStream_t st) {
    const int chunk_tokens = chunk_tokens_for(max_seq_len);
    const int n_chunks = max(1, (max_seq_len + chunk_tokens - 1) / chunk_tokens);
    dim3 grid(n_chunks, Hkv, B);
    scan_hist_kernel<G><<<grid, kScanThreads, 0, st>>>(q_codes, k_codes, kc_sb, kc_sh, seq_lens, max_seq_len,
                                                      Hq, Hkv, chunk_tokens, ws_hist);
    select_kernel<G><<<grid, kScanThreads, 0, st>>>(q_codes, k_codes, kc_sb, kc_sh, seq_lens, max_seq_len, k_per_seq,
                                                   k_uniform, k_max, Hq, Hkv, chunk_tokens, ws_hist, idx, idx_sb, idx_sh,
                                                   count, hist_out);
    count_launch(2);
    return cudaGetLastError();
}

cudaError_t launch_score_topk(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes,
                              long long kc_sb, long long kc_sh, const int32_t *seq_lens,
                              const int32_t *k_per_seq, int k_uniform, int max_seq_len, int k_max,
                              int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                              int32_t *hist_out, int32_t *ws_hist, cudaStream_t st) {
#define HA_ARGS B, Hq, Hkv, q_codes, k_codes, kc_sb, kc_sh, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx, \
                idx_sb, idx_sh, count, hist_out, ws_hist, st
    switch (Hq / Hkv) {
        case 1: return launch_g<1>(HA_ARGS);
        case 2: return launch_g<2>(HA_ARGS);
        case 4: return launch_g<4>(HA_ARGS);
        case 8: return launch_g<8>(HA_ARGS);
        default: return cudaErrorInvalidValue;
    }
#undef HA_ARGS
}

} // namespace ha
