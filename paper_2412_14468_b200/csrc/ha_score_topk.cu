// SCORE + TOPK.  Scores are s = 32 - popc(k_code ^ q_code) (Eq. 1 via the bitcount-xor identity of
// Section 4.1), reduced with max over the query heads of the GQA group, so they take only 33
// values.  "Standard top-k" (Section 4) therefore needs no sort: a histogram gives the threshold
// score T and how many tokens r of score exactly T are still needed; the selection is every token
// above T plus the first r tokens at T in index order, written in ascending token order.
//
// Two implementations share the arithmetic:
//  * sequences of up to 131072 tokens: ONE kernel, a thread-block cluster per (sequence, KV head)
//    (score_select_cluster_kernel, second half of this file);
//  * longer sequences: two kernels over chunks of the sequence, with the per-chunk histograms and
//    one score byte per token passed through the workspace (scan_score_kernel, select_kernel).
// No CTA ever spins on another: hand-offs are hardware cluster barriers or kernel boundaries.
// The scanning kernels request their first signatures before the programmatic-launch wait, so that
// the fetch overlaps the tail of the preceding kernel; the one signature that the preceding ENCODE
// may still be writing (the appended token, slot n-1) is re-read after the wait.
#include <cstdlib>
#include "ha_score_dev.cuh"

namespace ha {

constexpr int kScanThreads = 256;
constexpr int kPassTokens = kScanThreads * 16;   // four uint4 per thread
constexpr int kClusterMaxSeq = 8 * 8 * 2048;     // longest sequence the cluster kernel takes (8 CTAs x 8 rows x 2048 tokens)

// ------------------------------------------------------------------ long-sequence path (two kernels)

// Kernel 1: one chunk per CTA.  Streams the chunk's signatures (four uint4 per thread in flight, the
// next pass requested before the current one is scored), leaves the group scores as one byte per
// token in the workspace (so that kernel 2 needs neither the signatures nor popc again) and the
// chunk's 33-bin histogram.  Counting: one 32-bit counter per (level, lane), shared by the warps and
// bumped with shared-memory reductions (a lane only meets its own column; nothing waits for a result).
template <int G>
__global__ void __launch_bounds__(kScanThreads) scan_score_kernel(const uint32_t *__restrict__ q_codes,
                                                                 const uint32_t *__restrict__ k_codes,
                                                                 long long kc_sb, long long kc_sh,
                                                                 const int32_t *__restrict__ seq_lens,
                                                                 int max_seq_len, int Hq, int Hkv,
                                                                 int chunk_tokens, long long score_row,
                                                                 unsigned char *__restrict__ ws_scores,
                                                                 int32_t *__restrict__ ws_hist, Windows win, CodePages cp,
                                                                 int row_shift) {
    __shared__ __align__(16) uint32_t c_hist[kBins][32];
    __shared__ int s_hist[kBins + 3];
    __shared__ uint32_t s_qc[G];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int kvh = row_shift >= 0 ? (g >> row_shift) : g;   // the KV head whose signatures this unit scans
    const bool paged = cp.table != nullptr;
    const int32_t *table_b = paged ? cp.table + (long long)b * cp.bt_sb : nullptr;
    const int n = min(seq_lens[b], max_seq_len);
    const int start = chunk * chunk_tokens;
    if (start >= n) return;
    const int tid = threadIdx.x, lane = tid & 31;
    // contiguous cache: the unit's row; paged cache: the pool from this head's offset on
    const uint32_t *row = paged ? k_codes + (long long)kvh * cp.head_stride : k_codes + (long long)b * kc_sb + (long long)kvh * kc_sh;
    uint32_t *srow = reinterpret_cast<uint32_t *>(ws_scores + ((long long)b * Hkv + g) * score_row);
    const int end = min(n, start + chunk_tokens);
    const WindowBounds wbd = window_bounds(win, n);   // always-kept tokens: byte kForcedByte, not counted

    // pass = 4096 tokens: sub-block j of 1024 tokens, one uint4 per thread (coalesced)
    auto load_pass = [&](uint4 (&c)[4], int pass) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int base = pass + j * 1024 + tid * 4;
            if (base >= end) c[j] = make_uint4(0, 0, 0, 0);
            else c[j] = paged ? load_codes4_paged(cp, row, table_b, base, end) : load_codes4(row, base, end);
        }
    };
    uint4 cur[4], nxt[4];
    load_pass(cur, start);
    for (int i = tid; i < kBins * 32 / 4; i += kScanThreads)
        reinterpret_cast<uint4 *>(&c_hist[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    if (tid < kBins + 3) s_hist[tid] = 0;
    pdl_launch_dependents();
    pdl_wait();
    // The query signatures were written by the kernel in front of this one and must come from L2; the many
    // CTAs of a long sequence all want the same few words, so one thread per word fetches them for the CTA.
    if (tid < G) s_qc[tid] = __ldcg(q_codes + (long long)b * Hq + g * G + tid);
    __syncthreads();
    uint32_t qc[G];
#pragma unroll
    for (int j = 0; j < G; ++j) qc[j] = s_qc[j];

    // the counter of score s sits (32 - s) rows below the lane's counter of level 32
    const uint32_t top = (uint32_t)__cvta_generic_to_shared(&c_hist[kBins - 1][lane]);
    auto bump = [&](int ham) { asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(top - (uint32_t)ham * 128u) : "memory"); };
    auto hamming = [&](uint32_t code) {
        int h = __popc(code ^ qc[0]);
#pragma unroll
        for (int j = 1; j < G; ++j) h = min(h, __popc(code ^ qc[j]));
        return h;
    };
    for (int pass = start; pass < end; pass += kPassTokens) {
        if (pass + kPassTokens < end) load_pass(nxt, pass + kPassTokens);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int base = pass + j * 1024 + tid * 4;
            if (base < end) {
                if (paged) {
                    patch_token_paged(cur[j], base, n - 1, cp, row, table_b);
                    patch_token_paged(cur[j], base, n - 2, cp, row, table_b);
                } else {
                    patch_token(cur[j], base, n - 1, row);   // the appended token may just have been written,
                    patch_token(cur[j], base, n - 2, row);   // and the one before it by a layer-step directly in front
                }
                const int h0 = hamming(cur[j].x), h1 = hamming(cur[j].y), h2 = hamming(cur[j].z), h3 = hamming(cur[j].w);
                // bytes 33 - h = score + 1 (0 = no token); no byte borrows because h <= 32
                uint32_t s4 = 0x21212121u - ((uint32_t)h0 | ((uint32_t)h1 << 8) | ((uint32_t)h2 << 16) | ((uint32_t)h3 << 24));
                if (base + 3 < end && base >= wbd.sink_end && base + 4 <= wbd.local_begin) {
                    bump(h0); bump(h1); bump(h2); bump(h3);   // whole uint4 inside the chunk, outside the windows
                } else {
                    const int hh[4] = {h0, h1, h2, h3};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int t = base + e;
                        if (t >= end) s4 &= ~(0xffu << (8 * e));                           // zero byte: no token
                        else if (t < wbd.sink_end || t >= wbd.local_begin) s4 = (s4 & ~(0xffu << (8 * e))) | (kForcedByte << (8 * e));
                        else bump(hh[e]);
                    }
                }
                srow[base >> 2] = s4;
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) cur[j] = nxt[j];
    }
    __syncthreads();
    for (int i = tid; i < kBins * 8; i += kScanThreads) {   // eight threads per level, four counters each
        const uint4 v = reinterpret_cast<const uint4 *>(&c_hist[i >> 3][0])[i & 7];
        const uint32_t ssum = (v.x + v.y) + (v.z + v.w);
        if (ssum) atomicAdd(&s_hist[i >> 3], (int)ssum);
    }
    __syncthreads();
    if (tid < kBins) ws_hist[(((long long)b * Hkv + g) * kMaxChunks + chunk) * kBins + tid] = s_hist[tid];
}

// Kernel 2: one chunk per CTA.  Sums the chunk histograms (total, and the part before its own
// chunk), derives T, r and its output offset, then walks its chunk's score bytes (16 consecutive
// tokens per thread and pass) and writes the selected token indices in ascending order.
__global__ void __launch_bounds__(kScanThreads) select_kernel(const int32_t *__restrict__ seq_lens, int max_seq_len,
                                                             const int32_t *__restrict__ k_per_seq, int k_uniform,
                                                             int k_max, int Hkv, int chunk_tokens, long long score_row,
                                                             const unsigned char *__restrict__ ws_scores,
                                                             const int32_t *__restrict__ ws_hist,
                                                             int32_t *__restrict__ idx, long long idx_sb,
                                                             long long idx_sh, int32_t *__restrict__ count,
                                                             int32_t *__restrict__ hist_out, Windows win) {
    __shared__ int s_wtot[kScanThreads / 32][kBins + 3], s_wbef[kScanThreads / 32][kBins + 3];
    __shared__ int warp_tot[kScanThreads / 32];
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = max(min(seq_lens[b], max_seq_len), 0);
    int k = k_per_seq ? k_per_seq[b] : k_uniform;
    const WindowBounds wbd = window_bounds(win, n);
    const int n_forced = forced_before(wbd, n);
    const int keep_rest = max(0, min(min(k, k_max - n_forced), n - n_forced));   // heavy tokens among the others
    const int keep = n_forced + keep_rest;
    const int n_chunks = (n + chunk_tokens - 1) / chunk_tokens;
    if (chunk > 0 && chunk >= n_chunks) return;
    pdl_launch_dependents();
    pdl_wait();   // histograms and score bytes come from the preceding kernel

    const uint4 *srow = reinterpret_cast<const uint4 *>(ws_scores + ((long long)b * Hkv + g) * score_row);
    const int start = chunk * chunk_tokens, end = min(n, start + chunk_tokens);
    // first pass of score bytes: requested now, used after the threshold is known
    uint4 sv_next = make_uint4(0u, 0u, 0u, 0u);
    if (chunk < n_chunks && start + tid * 16 < end) sv_next = __ldcg(srow + ((start + tid * 16) >> 4));

    // totals per score level, and the part contributed by the chunks before this one.  Lane l of warp w sums
    // level l over the chunks w, w + 8, ... (coalesced rows of the counter table, every load issued before
    // the first use), lane 0 also level 32; the eight warps' sums meet in shared memory.  No atomics: a
    // hundred adds queued on one shared-memory word would stall the loads that follow them.
    {
        const int32_t *hb = ws_hist + ((long long)b * Hkv + g) * kMaxChunks * kBins;
        constexpr int kWarps = kScanThreads / 32, kPer = kMaxChunks / kWarps;
        int v[kPer], v32[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int cc = warp + i * kWarps;
            v[i] = (cc < n_chunks) ? __ldcg(hb + cc * kBins + lane) : 0;
            v32[i] = (cc < n_chunks && lane == 0) ? __ldcg(hb + cc * kBins + 32) : 0;
        }
        int tot = 0, bef = 0, tot32 = 0, bef32 = 0;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int cc = warp + i * kWarps;
            tot += v[i];
            tot32 += v32[i];
            if (cc < chunk) { bef += v[i]; bef32 += v32[i]; }
        }
        s_wtot[warp][lane] = tot;
        s_wbef[warp][lane] = bef;
        if (lane == 0) { s_wtot[warp][32] = tot32; s_wbef[warp][32] = bef32; }
    }
    __syncthreads();
    // Every warp folds the eight partial sums and derives the threshold for itself (lane l owns level l,
    // level 32 is read by every lane): no broadcast, no further barrier.  Suffix sums over the levels give
    // #{S >= t}; T = largest level with #{S >= T} >= keep; r = keep - #{S > T}.
    int T, r, gt_before, eq_before;
    {
        int tot = 0, bef = 0, tot32 = 0, bef32 = 0;
#pragma unroll
        for (int w = 0; w < kScanThreads / 32; ++w) {
            tot += s_wtot[w][lane];
            bef += s_wbef[w][lane];
            tot32 += s_wtot[w][32];
            bef32 += s_wbef[w][32];
        }
        find_threshold(tot, bef, tot32, bef32, keep_rest, lane, T, r, gt_before, eq_before);
        if (warp == 0 && chunk == 0 && hist_out) {
            hist_out[((long long)b * Hkv + g) * kBins + lane] = tot;
            if (lane == 0) hist_out[((long long)b * Hkv + g) * kBins + 32] = tot32;
        }
    }
    int32_t *out = idx + (long long)b * idx_sb + (long long)g * idx_sh;
    if (chunk == 0) {
        if (tid == 0) count[b * Hkv + g] = keep;
        for (int i = keep + tid; i < k_max; i += kScanThreads) out[i] = -1;
    }
    if (chunk >= n_chunks || keep == 0) return;

    // Per byte b = score + 1 (0 = no token): b + 127 - (T+1) sets bit 7 iff score > T, b + 128 - (T+1) iff
    // score >= T (no byte sum reaches 256).
    const uint32_t T4 = (uint32_t)(T + 1) * 0x01010101u;
    const uint32_t c_gt = 0x7f7f7f7fu - T4, c_ge = 0x80808080u - T4;
    // tokens before this pass with S > T (always-kept tokens count as such) / S == T
    int run_gt = gt_before + forced_before(wbd, start), run_eq = eq_before;
    for (int pass = start; pass < end; pass += kPassTokens) {
        const int base = pass + tid * 16;
        const uint4 sv = sv_next;
        sv_next = make_uint4(0u, 0u, 0u, 0u);
        if (base + kPassTokens < end) sv_next = __ldcg(srow + ((base + kPassTokens) >> 4));   // next pass, in flight
        const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w};
        uint32_t gt16 = 0u, ge16 = 0u;   // bit i = token base + i
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // words past the chunk were never written: drop them (end is a multiple of 4 or the sequence end)
            const uint32_t w = (base + 4 * j < end) ? sw[j] : 0u;
            gt16 |= high_bits_to_nibble(w + c_gt) << (4 * j);
            ge16 |= high_bits_to_nibble(w + c_ge) << (4 * j);
        }
        const uint32_t eq16 = ge16 ^ gt16;   // score > T implies score >= T
        const int packed = __popc(gt16) | (__popc(eq16) << 16);
        // block-wide exclusive prefix of the packed (gt, eq) counts (a pass has 4096 tokens: 16-bit halves suffice)
        int inc = packed;
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, dd);
            if (lane >= dd) inc += v;
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
        if (packed != 0) {
            const int excl = wpre + inc - packed;
            int g_run = run_gt + (excl & 0xffff);
            int q_run = run_eq + (int)((unsigned)excl >> 16);
            write_selected32(out, base, gt16, eq16, g_run, q_run, r);
        }
        run_gt += all & 0xffff;
        run_eq += (int)((unsigned)all >> 16);
        __syncthreads();   // warp_tot is rewritten by the next pass
    }
}

// ------------------------------------------------------------------ fused single-kernel path
//
// For sequences of up to CS * 16384 tokens one thread-block cluster of CS = 8, 4 or 2 CTAs owns a
// (sequence, KV head) unit: every CTA leaves the scores of its slice in shared memory (one byte per
// token), the CTAs exchange their 33-bin histograms through distributed shared memory between two
// hardware cluster barriers, and each CTA then compacts its own slice from those bytes.  The
// signatures are read from HBM once, there is no histogram round trip through global memory and no
// second launch.
// Reading: a warp owns 256*Rb consecutive tokens and reads them in rows of 256 tokens, a lane 8
// consecutive tokens (one 32-byte sector) per row, so that every request of a warp covers 1 KB of
// contiguous memory.  Few registers are live (no per-thread score array), so six CTAs share an SM
// and hide each other's barriers and the latency of the population-count unit, which is the
// scarce resource here (one quarter-rate instruction per query head and token).
// Counting: one 32-bit counter per (level, lane), shared by the eight warps and bumped with
// shared-memory reductions: a lane only meets its own column, so an instruction never conflicts
// with itself, and nothing waits for a result.
// Writing: lane l owns the 8*Rb consecutive tokens l*8*Rb .. of its warp's range, so the prefix sums
// need one warp-shuffle scan plus one exchange of eight warp totals; only flagged tokens are
// visited, with plain integer arithmetic (the selection never queues behind the scoring for the
// population-count unit).

constexpr int kClusterMaxRows = 8;   // rows of 8 tokens per lane: a lane's flags fit one 64-bit word each

template <int G, int CS>
__global__ void __launch_bounds__(kScanThreads, 6) score_select_cluster_kernel(
    const uint32_t *__restrict__ q_codes, const uint32_t *__restrict__ k_codes, long long kc_sb, long long kc_sh,
    const int32_t *__restrict__ seq_lens, int max_seq_len, const int32_t *__restrict__ k_per_seq, int k_uniform,
    int k_max, int Hq, int Hkv, int32_t *__restrict__ idx, long long idx_sb, long long idx_sh,
    int32_t *__restrict__ count, int32_t *__restrict__ hist_out, Windows win) {
    extern __shared__ __align__(16) unsigned char s_sc[];      // score + 1 of this CTA's tokens (0 = no token)
    __shared__ __align__(16) uint32_t c_hist[kBins][32];       // counters [level][lane]
    __shared__ int s_hist[kBins + 3];          // this CTA's histogram, read by the whole cluster
    __shared__ int s_tot[kBins], s_bef[kBins];
    __shared__ int sh_T, sh_r, sh_gt_before, sh_eq_before;
    __shared__ int s_wcnt[kScanThreads / 32];
    const uint32_t rank = cluster_rank();
    const int g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = max(min(seq_lens[b], max_seq_len), 0);
    int k = k_per_seq ? k_per_seq[b] : k_uniform;
    const WindowBounds wbd = window_bounds(win, n);   // always-kept tokens: byte kForcedByte, not counted
    const int n_forced = forced_before(wbd, n);
    const int keep_rest = max(0, min(min(k, k_max - n_forced), n - n_forced));   // heavy tokens among the others
    const int keep = n_forced + keep_rest;
    const uint32_t *row = k_codes + (long long)b * kc_sb + (long long)g * kc_sh;
    // The sequence's own length is divided over the CS CTAs (ragged batches stay balanced): Rb rows per
    // lane, a warp owns the 256*Rb tokens from wb on, a CTA 2048*Rb; row p of a lane is
    // wb + 256 p + 8 lane .. + 7.
    const int Rb = (n + CS * 2048 - 1) / (CS * 2048);
    const int wl = warp * 256 * Rb;                    // the warp's first token inside the CTA's slice
    const int wb = (int)rank * 2048 * Rb + wl;

    auto load_row = [&](int p, uint4 &lo, uint4 &hi, bool early) {
        const int t = wb + p * 256 + lane * 8;
        if (p < Rb && t + 8 <= n) {
            const uint4 *src = reinterpret_cast<const uint4 *>(row + t);
            if (early) { lo = __ldg(src); hi = __ldg(src + 1); }
            else { lo = __ldcg(src); hi = __ldcg(src + 1); }
        } else {
            lo = (p < Rb && t < n) ? load_codes4(row, t, n) : make_uint4(0, 0, 0, 0);
            hi = (p < Rb && t + 4 < n) ? load_codes4(row, t + 4, n) : make_uint4(0, 0, 0, 0);
        }
    };
    uint4 c[4];   // two rows
    load_row(0, c[0], c[1], true);
    load_row(1, c[2], c[3], true);
    // the other rows of this warp start their way from HBM to L2 now (one request per 128-byte line, no registers): the
    // loads that follow turn by turn then wait for L2 only, which is what counts when few CTAs share the SM
    for (int p = 2; p < Rb; ++p) {
        const int t = wb + p * 256 + lane * 8;
        if ((lane & 3) == 0 && t < n) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + t));
    }
    for (int i = tid; i < kBins * 32 / 4; i += kScanThreads)
        reinterpret_cast<uint4 *>(&c_hist[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    if (tid < kBins + 3) s_hist[tid] = 0;
    pdl_launch_dependents();
    pdl_wait();
    // the signatures that a library kernel directly in front may just have written (slot n-1 by ENCODE, slot n-2
    // by a layer-step for the sequence one token shorter): re-read by the one lane that holds them
#pragma unroll
    for (int back = 1; back <= 2; ++back) {
        const int e_last = (n - back) - wb;
        if (e_last >= 0 && e_last < 512 && e_last < 256 * Rb && ((e_last & 255) >> 3) == lane) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                patch_token(c[2 * j], wb + j * 256 + lane * 8, n - back, row);
                patch_token(c[2 * j + 1], wb + j * 256 + lane * 8 + 4, n - back, row);
            }
        }
    }
    uint32_t qc[G];
#pragma unroll
    for (int j = 0; j < G; ++j) qc[j] = __ldcg(q_codes + (long long)b * Hq + g * G + j);
    __syncthreads();

    // ---- scores (four score+1 bytes per word) and this CTA's histogram.  The counter of score s sits
    // (32 - s) rows below the lane's counter of level 32, so the address comes straight from the
    // Hamming distance 32 - s.
    const uint32_t top = (uint32_t)__cvta_generic_to_shared(&c_hist[kBins - 1][lane]);
    auto bump = [&](int ham) { asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(top - (uint32_t)ham * 128u) : "memory"); };
    auto hamming = [&](uint32_t code) {
        int h = __popc(code ^ qc[0]);
#pragma unroll
        for (int j = 1; j < G; ++j) h = min(h, __popc(code ^ qc[j]));
        return h;
    };
    auto score_word = [&](const uint4 &cw, int t, bool whole_row) -> uint32_t {
        const int h0 = hamming(cw.x), h1 = hamming(cw.y), h2 = hamming(cw.z), h3 = hamming(cw.w);
        // bytes 33 - h = score + 1; no byte borrows because h <= 32
        uint32_t s4 = 0x21212121u - ((uint32_t)h0 | ((uint32_t)h1 << 8) | ((uint32_t)h2 << 16) | ((uint32_t)h3 << 24));
        if (whole_row) {
            bump(h0); bump(h1); bump(h2); bump(h3);
        } else {
            const int hh[4] = {h0, h1, h2, h3};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int tt = t + e;
                if (tt >= n) s4 &= ~(0xffu << (8 * e));                                // zero byte: no token
                else if (tt < wbd.sink_end || tt >= wbd.local_begin) s4 = (s4 & ~(0xffu << (8 * e))) | (kForcedByte << (8 * e));
                else bump(hh[e]);
            }
        }
        return s4;
    };
    for (int p0 = 0; p0 < Rb; p0 += 2) {   // CTA-uniform
        if (p0 > 0) {
            load_row(p0, c[0], c[1], false);
            load_row(p0 + 1, c[2], c[3], false);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int p = p0 + j, t = wb + p * 256 + lane * 8;
            if (p < Rb) {
                const bool whole_row = t + 8 <= n && t >= wbd.sink_end && t + 8 <= wbd.local_begin;
                uint2 w;
                w.x = score_word(c[2 * j], t, whole_row);
                w.y = score_word(c[2 * j + 1], t + 4, whole_row);
                *reinterpret_cast<uint2 *>(s_sc + wl + p * 256 + lane * 8) = w;
            }
        }
    }
    __syncthreads();
    // fold the counters: eight threads per level, four counters each
    for (int i = tid; i < kBins * 8; i += kScanThreads) {
        const uint4 v = reinterpret_cast<const uint4 *>(&c_hist[i >> 3][0])[i & 7];
        const uint32_t ssum = (v.x + v.y) + (v.z + v.w);
        if (ssum) atomicAdd(&s_hist[i >> 3], (int)ssum);
    }
    cluster_sync_all();   // every CTA's histogram is complete and visible cluster-wide

    if (tid < kBins) {
        int tot = 0, bef = 0;
#pragma unroll
        for (uint32_t r = 0; r < (uint32_t)CS; ++r) {
            const int v = ld_dsmem(&s_hist[tid], r);
            tot += v;
            if (r < rank) bef += v;
        }
        s_tot[tid] = tot;
        s_bef[tid] = bef;
    }
    // this CTA is done reading its peers' shared memory; the matching wait sits at the end of the
    // kernel, so that no CTA exits while a peer may still read its histogram
    cluster_arrive();
    __syncthreads();
    if (warp == 0) {
        int tot = s_tot[lane], bef = s_bef[lane];
        const int tot32 = s_tot[32], bef32 = s_bef[32];
        int T, r, gt_before, eq_before;
        find_threshold(tot, bef, tot32, bef32, keep_rest, lane, T, r, gt_before, eq_before);
        if (lane == 0) { sh_T = T; sh_r = r; sh_gt_before = gt_before; sh_eq_before = eq_before; }
        if (rank == 0 && hist_out) {
            hist_out[((long long)b * Hkv + g) * kBins + lane] = tot;
            if (lane == 0) hist_out[((long long)b * Hkv + g) * kBins + 32] = tot32;
        }
    }
    __syncthreads();
    const int T = sh_T, r = sh_r;
    int32_t *out = idx + (long long)b * idx_sb + (long long)g * idx_sh;
    if (rank == 0) {
        if (tid == 0) count[b * Hkv + g] = keep;
        for (int i = keep + tid; i < k_max; i += kScanThreads) out[i] = -1;
    }
    if (keep == 0) { cluster_wait(); return; }

    // ---- flags "S > T" / "S == T" of the lane's 8*Rb consecutive tokens (bit i = token first + i)
    // Per byte b = score + 1 (0 = no token): b + 127 - (T+1) sets bit 7 iff score > T, b + 128 - (T+1) iff
    // score >= T (no byte sum reaches 256); high_bits_to_nibble gathers the four bit-7 flags of a word.
    const uint32_t T4 = (uint32_t)(T + 1) * 0x01010101u;
    const uint32_t c_gt = 0x7f7f7f7fu - T4, c_ge = 0x80808080u - T4;
    const int first_l = wl + 8 * Rb * lane;
    uint32_t gt_lo = 0u, gt_hi = 0u, ge_lo = 0u, ge_hi = 0u;
#pragma unroll
    for (int j = 0; j < kClusterMaxRows; ++j) {
        if (j < Rb) {
            const uint2 w = *reinterpret_cast<const uint2 *>(s_sc + first_l + 8 * j);
            const uint32_t gb = high_bits_to_nibble(w.x + c_gt) | (high_bits_to_nibble(w.y + c_gt) << 4);
            const uint32_t eb = high_bits_to_nibble(w.x + c_ge) | (high_bits_to_nibble(w.y + c_ge) << 4);
            if (j < 4) { gt_lo |= gb << (8 * j); ge_lo |= eb << (8 * j); }
            else { gt_hi |= gb << (8 * (j - 4)); ge_hi |= eb << (8 * (j - 4)); }
        }
    }
    const uint32_t eq_lo = ge_lo ^ gt_lo, eq_hi = ge_hi ^ gt_hi;   // score > T implies score >= T
    const int tot_packed = (__popc(gt_lo) + __popc(gt_hi)) | ((__popc(eq_lo) + __popc(eq_hi)) << 16);
    int winc = tot_packed;   // inclusive scan over the lanes of the per-lane totals
#pragma unroll
    for (int dd = 1; dd < 32; dd <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, winc, dd);
        if (lane >= dd) winc += v;
    }
    if (lane == 31) s_wcnt[warp] = winc;
    __syncthreads();
    // tokens before this warp's range with S > T (always-kept tokens count as such) / S == T
    int run_gt = sh_gt_before + forced_before(wbd, min((int)rank * 2048 * Rb, n)), run_eq = sh_eq_before;
#pragma unroll
    for (int w = 0; w < kScanThreads / 32; ++w) {
        if (w < warp) { run_gt += s_wcnt[w] & 0xffff; run_eq += (int)((unsigned)s_wcnt[w] >> 16); }
    }
    if (tot_packed != 0) {
        const int excl = winc - tot_packed;
        int g_run = run_gt + (excl & 0xffff);
        int q_run = run_eq + (int)((unsigned)excl >> 16);
        const int first = (int)rank * 2048 * Rb + first_l;
        write_selected32(out, first, gt_lo, eq_lo, g_run, q_run, r);
        write_selected32(out, first + 32, gt_hi, eq_hi, g_run, q_run, r);
    }
    cluster_wait();
}

template <int G, int CS>
static cudaError_t launch_cluster_t(int rows, int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes,
                                    long long kc_sb, long long kc_sh, const int32_t *seq_lens,
                                    const int32_t *k_per_seq, int k_uniform, int max_seq_len, int k_max, int32_t *idx,
                                    long long idx_sb, long long idx_sh, int32_t *count, int32_t *hist_out,
                                    cudaStream_t st, Windows win) {
    static bool opted[64] = {};   // opt in to the padded shared-memory sizes once per device
    {
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev >= 0 && dev < 64 && !opted[dev]) {
            cudaError_t e = cudaFuncSetAttribute(score_select_cluster_kernel<G, CS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
            if (e != cudaSuccess) return e;
            opted[dev] = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS, Hkv, B);
    cfg.blockDim = dim3(kScanThreads);
    cfg.dynamicSmemBytes = (size_t)rows * 2048;   // one score byte per token of the CTA's slice (<= 16 KB)
    {
        // Launched behind another kernel, the CTAs land wherever room appears first, and an SM that takes six of them
        // while others hold two sets the kernel's time (the population-count unit is shared by the CTAs of an SM).
        // When the grid needs fewer than six CTAs per SM, shared memory is requested as if each CTA needed a whole
        // share of the SM, so that no SM can take more than ceil(CTAs / SMs).  Clusters of 4 or 8 need some slack
        // for that (all CTAs of a cluster are placed together): without it the cap only delays their placement.
        const int n_ctas = CS * Hkv * B, n_sm = sm_count();
        const int cap = (n_ctas + n_sm - 1) / n_sm;   // CTAs per SM
        const bool slack = CS == 2 || 2 * (cap * n_sm - n_ctas) >= n_sm;
        if (n_ctas > n_sm && cap < 6 && slack) {
            static size_t pad[64][6] = {};   // per device and cap: the least dynamic shared memory with which only `cap` CTAs fit
            int dev = 0;
            cudaGetDevice(&dev);
            if (dev < 0 || dev >= 64) dev = 0;
            if (!pad[dev][cap]) {
                size_t found = 0;
                for (size_t kb = 8; kb <= 100 && !found; ++kb) {
                    int occ = 0;
                    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, score_select_cluster_kernel<G, CS>, kScanThreads, kb * 1024) != cudaSuccess) break;
                    if (occ <= cap) found = kb * 1024;
                }
                pad[dev][cap] = found ? found : 1;
            }
            if (pad[dev][cap] > cfg.dynamicSmemBytes) cfg.dynamicSmemBytes = pad[dev][cap];
        }
    }
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, score_select_cluster_kernel<G, CS>, q_codes, k_codes, kc_sb, kc_sh,
                                       seq_lens, max_seq_len, k_per_seq, k_uniform, k_max, Hq, Hkv, idx, idx_sb, idx_sh,
                                       count, hist_out, win);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

template <int G>
static cudaError_t launch_g(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes,
                            long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq,
                            int k_uniform, int max_seq_len, int k_max, int32_t *idx, long long idx_sb,
                            long long idx_sh, int32_t *count, int32_t *hist_out, int32_t *ws_hist,
                            unsigned char *ws_scores, cudaStream_t st, Windows win, CodePages cp, int row_shift) {
    if (max_seq_len <= kClusterMaxSeq && !cp.table && row_shift < 0) {
        // Fused path: one cluster per unit.  Cluster size: the largest of 8, 4, 2 whose grid still fits
        // the GPU in one wave (about six 256-thread CTAs per SM), so that small batches get the most
        // parallelism per sequence and large batches the most work per cluster barrier; a lane then
        // holds R = ceil(n / (CS * 2048)) rows of 8 tokens (R <= 8).
        const int units = B * Hkv, one_wave = 6 * sm_count();
        int cs = 8;
        while (cs > 2 && units * cs > one_wave) cs >>= 1;
        while ((max_seq_len + cs * 2048 - 1) / (cs * 2048) > kClusterMaxRows) cs <<= 1;
        const int rows = max(1, (max_seq_len + cs * 2048 - 1) / (cs * 2048));
#define HA_CL(CSZ)                                                                                                    \
    return launch_cluster_t<G, CSZ>(rows, B, Hq, Hkv, q_codes, k_codes, kc_sb, kc_sh, seq_lens, k_per_seq, k_uniform, \
                                    max_seq_len, k_max, idx, idx_sb, idx_sh, count, hist_out, st, win)
        if (cs == 8) HA_CL(8);
        if (cs == 4) HA_CL(4);
        HA_CL(2);
#undef HA_CL
    }
    const int chunk_tokens = chunk_tokens_for(B * Hkv, max_seq_len, sm_count());
    const int n_chunks = max(1, (max_seq_len + chunk_tokens - 1) / chunk_tokens);
    const long long score_row = (long long)score_row_bytes(max_seq_len);
    dim3 grid(n_chunks, Hkv, B);
    cudaError_t e = launch_pdl(scan_score_kernel<G>, grid, dim3(kScanThreads), 0, st, q_codes, k_codes, kc_sb, kc_sh,
                               seq_lens, max_seq_len, Hq, Hkv, chunk_tokens, score_row, ws_scores, ws_hist, win, cp, row_shift);
    if (e != cudaSuccess) return e;
    e = launch_pdl(select_kernel, grid, dim3(kScanThreads), 0, st, seq_lens, max_seq_len, k_per_seq, k_uniform, k_max,
                   Hkv, chunk_tokens, score_row, (const unsigned char *)ws_scores, (const int32_t *)ws_hist, idx, idx_sb,
                   idx_sh, count, hist_out, win);
    if (e != cudaSuccess) return e;
    count_launch(2);
    return cudaGetLastError();
}

cudaError_t launch_score_topk(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes,
                              long long kc_sb, long long kc_sh, const int32_t *seq_lens,
                              const int32_t *k_per_seq, int k_uniform, int max_seq_len, int k_max,
                              int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                              int32_t *hist_out, int32_t *ws_hist, unsigned char *ws_scores, cudaStream_t st, Windows win,
                              CodePages cp, int row_shift) {
    if (row_shift >= 0) {   // one unit per query head: groups of one head over Hq unit heads
        return launch_g<1>(B, Hq, Hq, q_codes, k_codes, kc_sb, kc_sh, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx, idx_sb,
                           idx_sh, count, hist_out, ws_hist, ws_scores, st, win, cp, row_shift);
    }
#define HA_ARGS B, Hq, Hkv, q_codes, k_codes, kc_sb, kc_sh, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx, \
                idx_sb, idx_sh, count, hist_out, ws_hist, ws_scores, st, win, cp, -1
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
