// SCORE + TOPK and GATHER-ATT of a layer-step in ONE persistent kernel, for steps with too many (sequence, KV head)
// units for the single-cluster kernel of ha_fused.cu (entry point ha_sparse_decode_pipelined; ha_sparse_decode itself runs
// such steps as three kernels, which is the faster schedule on B200: see the note on scoring further down).
//
// Why: at scale the two halves of the step are bound by different units of the SM.  SCORE (Eq. 1 as bitcount(xor),
// Section 4.1) spends its time in the population-count pipe and the integer pipe; GATHER-ATT (Section 4) waits for
// HBM.  Run one after the other, each leaves the other's resource idle.  Here every SM holds one CTA of 28 warps
// with two roles (the register file is re-divided between them with setmaxnreg: 40 registers per SCORE thread, 152
// per GATHER thread, out of the 72 per thread the CTA is launched with):
//   * twenty SCORE warps walk the units of the CTA's range: scores as one byte per token, a histogram per group of
//     four warps, the threshold of the standard top-k (Section 4), the index list in ascending token order (ties to
//     the lowest index), then a release counter per unit;
//   * eight GATHER warps follow them over the same range: each warp keeps a two-stage ring of 16-row blocks in flight
//     (16-byte cp.async, a half-warp per 256-byte row), waits for a unit's counter before it touches the unit's list,
//     and keeps requesting rows of the next unit while the states of the previous one are merged, so that the row
//     stream never drains inside a CTA's range.
// Work split: the 16-entry blocks of all index lists, laid end to end, are cut into equal contiguous ranges, one per
// CTA (list lengths are min(k, n) + the always-kept windows, known before anything is scored).  A unit that lies
// inside one range is scored by that CTA; a unit that several ranges share is scored by those CTAs together, one
// chunk of the sequence each: chunk histograms meet in the workspace, every CTA derives the same threshold, and the
// scores of such a chunk wait in the workspace (one byte per token) between the two passes.  Each CTA scores the
// chunks of its shared units FIRST, so that no CTA ever waits for another one's whole range.
// Waiting: a wait polls a counter in global memory that another CTA's SCORE warps (or its own) bump; SCORE warps
// never wait for GATHER warps, a chunk's first pass never waits at all, and all CTAs are resident at once (one per
// SM), so every wait ends.  Every wait is bounded all the same: when it runs out the kernel raises HA_DEV_TIMEOUT
// in the status word, sets an abort word that ends all other waits, and runs to its end without faulting (list
// entries are range-checked), leaving outputs that must not be used.
#include "ha_attn_dev.cuh"
#include "ha_score_dev.cuh"

namespace ha {

constexpr int kPipeGatherWarps = 8;
constexpr int kPipeScoreWarps = 20;
constexpr int kPipeScoreGroups = 5;                   // counter tables: one per four SCORE warps
constexpr int kPipeGatherRegs = 152, kPipeScoreRegs = 40;   // per thread once the roles part (setmaxnreg): 8 x 32 x 152 + 20 x 32 x 40 = 896 x 72, exactly what the CTA is launched with (a role can only take what the other gave back)
constexpr int kPipeGatherThreads = kPipeGatherWarps * 32;
constexpr int kPipeScoreThreads = kPipeScoreWarps * 32;
constexpr int kPipeThreads = kPipeGatherThreads + kPipeScoreThreads;
constexpr int kPipeStages = 2;                         // row blocks in flight per gather warp
constexpr int kPipeWarpRing = kPipeStages * kStageBytes;
constexpr int kPipeRingBytes = kPipeGatherWarps * kPipeWarpRing;
constexpr int kPipeLocalTokens = 32768;                // score bytes of one chunk that fit in shared memory
constexpr int kPipeHistBytes = kPipeScoreGroups * kBins * 32 * 4;
constexpr int kPipePrefBytes = (kMaxBalancedUnits + 4) * 4;
constexpr int kPipeCntStride = 36;
constexpr int kPipeSpinLimit = 1 << 22;                // polls of ~0.25 us each before a wait gives up

__host__ __device__ constexpr int pipe_scratch_bytes(int G) { return kPipeGatherWarps * G * kD * 4; }
__host__ __device__ constexpr int pipe_smem_bytes(int G) {
    return kPipeRingBytes + pipe_scratch_bytes(G) + kPipeLocalTokens + kPipeHistBytes + kPipePrefBytes;
}

struct PipeArgs {
    // SCORE + TOPK
    const uint32_t *q_codes, *k_codes;
    long long kc_sb, kc_sh;
    const int32_t *seq_lens, *k_per_seq;
    int k_uniform, max_seq_len, k_max;
    Windows win;
    int32_t *idx;
    long long idx_sb, idx_sh;
    int32_t *count;
    // GATHER-ATT
    const uint16_t *q;
    TensorView K, V;
    const int32_t *block_table;
    long long bt_sb;
    int page_shift, page_rows;
    float scale_log2;
    uint16_t *out;
    float *lse;
    int Hq, Hkv, n_units;
    // scratch (caller's workspace)
    int32_t *tickets, *s1_done, *s2_done;   // [n_units] each, zero between calls
    int32_t *ws_hist;                       // [n_units][kMaxChunks][33]
    unsigned char *ws_scores;               // [n_units][score_row]
    long long score_row;
    float *part_ml, *part_acc;
    uint32_t *status;                       // word 0: device status, word 1: abort
};

__device__ __forceinline__ int ld_acquire(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void bar_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }

// A wait that ran out: raise HA_DEV_TIMEOUT, end all other waits (abort word) and leave a note for a debugger in
// words 2.. of the workspace header (which wait, CTA, unit, awaited value, value seen).
__device__ __forceinline__ void pipe_give_up(uint32_t *status, int which, int unit, int want, int seen) {
    if (atomicExch(status + 1, 1u) == 0u) {
        status[2] = (uint32_t)which; status[3] = blockIdx.x; status[4] = (uint32_t)unit; status[5] = (uint32_t)want;
        status[6] = (uint32_t)seen; status[7] = threadIdx.x;
    }
    atomicOr(status, HA_DEV_TIMEOUT);
}

// Polls *counter until it reaches `want`.  Returns false when the wait was given up (its own limit, or another
// waiter's: the abort word); the caller then carries on with whatever is in memory.
__device__ __forceinline__ bool pipe_wait(const int32_t *counter, int want, uint32_t *status, bool &gave_up, int which, int unit) {
    if (gave_up) return false;
    int seen = 0;
    for (int it = 0; it < kPipeSpinLimit; ++it) {
        seen = ld_acquire(counter);
        if (seen >= want) return true;
        if ((it & 63) == 63 && ld_acquire(reinterpret_cast<const int32_t *>(status + 1)) != 0) { gave_up = true; return false; }
        __nanosleep(it < 64 ? 40 : 250);
    }
    gave_up = true;
    pipe_give_up(status, which, unit, want, seen);
    return false;
}

// Everything both roles derive from a unit's sequence length and budget.
struct PipeUnit {
    int b, kvh, n, keep, keep_rest;
    WindowBounds wbd;
};
__device__ __forceinline__ PipeUnit pipe_unit(const PipeArgs &a, int u) {
    PipeUnit r;
    r.b = u / a.Hkv;
    r.kvh = u - r.b * a.Hkv;
    r.n = max(min(a.seq_lens[r.b], a.max_seq_len), 0);
    const int k = a.k_per_seq ? a.k_per_seq[r.b] : a.k_uniform;
    r.wbd = window_bounds(a.win, r.n);
    const int nf = forced_before(r.wbd, r.n);
    r.keep_rest = max(0, min(min(k, a.k_max - nf), r.n - nf));
    r.keep = nf + r.keep_rest;
    return r;
}

// Which CTAs share unit u (blocks [u_lo, u_hi) of the global block sequence of T blocks cut into Pe ranges).
struct PipeSplit {
    int c_first, n_parts;
};
__device__ __forceinline__ PipeSplit pipe_split(long long u_lo, long long u_hi, long long T, long long Pe) {
    PipeSplit s;
    s.c_first = (int)(((u_lo + 1) * Pe - 1) / T);
    s.n_parts = (int)((u_hi * Pe - 1) / T) - s.c_first + 1;
    return s;
}
// Chunks of the sequence that the CTAs of a shared unit score: chunk c by part c.
__device__ __forceinline__ int pipe_chunks(int n, int n_parts) { return max(1, min(min(n_parts, kMaxChunks), (n + 1023) / 1024)); }
__device__ __forceinline__ int pipe_chunk_tokens(int n, int chunks) { return ((n + chunks - 1) / chunks + 1023) / 1024 * 1024; }

// ------------------------------------------------------------------ SCORE role

struct ScoreJob {
    int u;
    int t0, t1;          // tokens of the unit that this CTA scores
    int chunk, chunks;   // its chunk index and the number of chunks of the unit
    bool shared;         // the unit is shared with other CTAs: histograms meet in the workspace
    bool local;          // score bytes in shared memory (else in the workspace)
};

// Scoring needs many warps: a warp issues about one instruction in twelve cycles here (dependent population counts,
// shared-memory reductions, loads), so the twenty SCORE warps of a CTA together keep the population-count pipe far busier
// than four did (and still less busy than the 48 warps per SM of the stand-alone kernel).  They get by with few registers (two rows of signatures in flight per warp), which leaves the
// register file to the GATHER warps.
template <int G>
struct ScoreRole {
    const PipeArgs &a;
    unsigned char *s_local;      // kPipeLocalTokens score bytes
    uint32_t *s_hist;            // [kPipeScoreGroups][33][32] counters: one table per group of four warps
    int *s_cnt;                  // [kPipeScoreGroups][kPipeCntStride] level counts per table
    int *s_wcnt;                 // [kPipeScoreWarps][2] numbers of tokens with S > T / S == T in each warp's slice
    int sw, lane;                // score warp 0..15
    bool gave_up = false;

    __device__ ScoreRole(const PipeArgs &a_, unsigned char *loc, uint32_t *hist, int *cnt, int *wcnt, int sw_, int lane_)
        : a(a_), s_local(loc), s_hist(hist), s_cnt(cnt), s_wcnt(wcnt), sw(sw_), lane(lane_) {}

    __device__ __forceinline__ unsigned char *bytes_of(const ScoreJob &j) const {
        // byte of token t at base[t - j.t0]
        return j.local ? s_local : a.ws_scores + (long long)j.u * a.score_row + j.t0;
    }
    // this warp's tokens inside the job: whole rows of 256 tokens from a 256-aligned start
    __device__ __forceinline__ void warp_range(const ScoreJob &j, int &w0, int &w1) const {
        const int len = max(j.t1 - j.t0, 0);
        const int per = ((len + kPipeScoreWarps - 1) / kPipeScoreWarps + 255) / 256 * 256;
        w0 = min(j.t1, j.t0 + sw * per);
        w1 = min(j.t1, w0 + per);
    }

    // Pass 1: score bytes (score + 1; 0 = no token; kForcedByte = always kept) and the level counts of the job.
    // Ends with the job's counts in s_cnt (valid after the role barrier inside).
    __device__ void pass1(const ScoreJob &j, const PipeUnit &pu) {
        const int grp = sw >> 2, st = sw * 32 + lane;
        for (int i = st; i < kPipeScoreGroups * kBins * 32; i += kPipeScoreThreads) s_hist[i] = 0u;
        bar_sync(2, kPipeScoreThreads);
        uint32_t *hist = s_hist + grp * kBins * 32;
        int w0, w1;
        warp_range(j, w0, w1);
        const int n = pu.n;
        const uint32_t *row = a.k_codes + (long long)pu.b * a.kc_sb + (long long)pu.kvh * a.kc_sh;
        unsigned char *sc = bytes_of(j);
        uint32_t qc[G];
#pragma unroll
        for (int h = 0; h < G; ++h) qc[h] = __ldcg(a.q_codes + (long long)pu.b * a.Hq + pu.kvh * G + h);
        const uint32_t top = (uint32_t)__cvta_generic_to_shared(hist + (kBins - 1) * 32 + lane);
        auto bump = [&](int ham) { asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(top - (uint32_t)ham * 128u) : "memory"); };
        auto hamming = [&](uint32_t code) {
            int h = __popc(code ^ qc[0]);
#pragma unroll
            for (int jh = 1; jh < G; ++jh) h = min(h, __popc(code ^ qc[jh]));
            return h;
        };
        auto score_word = [&](const uint4 &cw, int t, bool whole) -> uint32_t {
            const int h0 = hamming(cw.x), h1 = hamming(cw.y), h2 = hamming(cw.z), h3 = hamming(cw.w);
            uint32_t s4 = 0x21212121u - ((uint32_t)h0 | ((uint32_t)h1 << 8) | ((uint32_t)h2 << 16) | ((uint32_t)h3 << 24));
            if (whole) {
                bump(h0); bump(h1); bump(h2); bump(h3);
            } else {
                const int hh[4] = {h0, h1, h2, h3};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int tt = t + e;
                    if (tt >= w1) s4 &= ~(0xffu << (8 * e));
                    else if (tt < pu.wbd.sink_end || tt >= pu.wbd.local_begin) s4 = (s4 & ~(0xffu << (8 * e))) | (kForcedByte << (8 * e));
                    else bump(hh[e]);
                }
            }
            return s4;
        };
        const int n_rows = (w1 - w0 + 255) / 256;
        auto load_row = [&](int r, uint4 &lo, uint4 &hi) {
            const int t = w0 + r * 256 + lane * 8;
            if (r < n_rows && t + 8 <= n) {
                const uint4 *src = reinterpret_cast<const uint4 *>(row + t);
                lo = __ldcg(src);
                hi = __ldcg(src + 1);
            } else {
                lo = (r < n_rows && t < n) ? load_codes4(row, t, n) : make_uint4(0, 0, 0, 0);
                hi = (r < n_rows && t + 4 < n) ? load_codes4(row, t + 4, n) : make_uint4(0, 0, 0, 0);
            }
        };
        uint4 c0, c1, n0, n1;   // the row being scored and the one behind it, requested a row ahead
        load_row(0, c0, c1);
        for (int r = 0; r < n_rows; ++r) {
            load_row(r + 1, n0, n1);
            const int t = w0 + r * 256 + lane * 8;
            const bool whole = t + 8 <= w1 && t >= pu.wbd.sink_end && t + 8 <= pu.wbd.local_begin;
            uint2 w;
            w.x = score_word(c0, t, whole);
            w.y = score_word(c1, t + 4, whole);
            *reinterpret_cast<uint2 *>(sc + (t - j.t0)) = w;
            c0 = n0; c1 = n1;
        }
        bar_sync(2, kPipeScoreThreads);
        // level counts per table: warp g folds table g (lane l adds the 32 counters of level l, rotated start: no bank conflict)
        if (sw < kPipeScoreGroups) {
            const uint32_t *hg = s_hist + sw * kBins * 32;
            int c = 0;
#pragma unroll 8
            for (int jj = 0; jj < 32; ++jj) c += (int)hg[lane * 32 + ((jj + lane) & 31)];
            int c32 = (int)hg[32 * 32 + lane];
#pragma unroll
            for (int dd = 16; dd > 0; dd >>= 1) c32 += __shfl_xor_sync(0xffffffffu, c32, dd);
            s_cnt[sw * kPipeCntStride + lane] = c;
            if (lane == 0) s_cnt[sw * kPipeCntStride + 32] = c32;
        }
        bar_sync(2, kPipeScoreThreads);
    }

    // level counts of the whole job (lane l: level l; level 32 in every lane)
    __device__ __forceinline__ void job_counts(int &tot, int &tot32) const {
        tot = 0; tot32 = 0;
#pragma unroll
        for (int w = 0; w < kPipeScoreGroups; ++w) { tot += s_cnt[w * kPipeCntStride + lane]; tot32 += s_cnt[w * kPipeCntStride + 32]; }
    }

    // Publishes the chunk's histogram (units shared by several CTAs).  All warps call it directly after pass1.
    __device__ void publish_chunk(const ScoreJob &j) {
        if (sw == 0) {
            int tot, tot32;
            job_counts(tot, tot32);
            int32_t *h = a.ws_hist + ((long long)j.u * kMaxChunks + j.chunk) * kBins;
            h[lane] = tot;
            if (lane == 0) h[32] = tot32;
        }
        // the score bytes of this chunk wait in the workspace: they and the histogram are visible before the counter moves
        __threadfence();
        bar_sync(2, kPipeScoreThreads);
        if (sw == 0 && lane == 0) atomicAdd(a.s1_done + j.u, 1);
    }

    // Pass 2: threshold, this warp's part of the index list, the unit's count and padding, release.
    __device__ void pass2(const ScoreJob &j, const PipeUnit &pu) {
        int w0, w1;
        warp_range(j, w0, w1);
        const unsigned char *sc = bytes_of(j);
        int tot, tot32, bef = 0, bef32 = 0;
        if (!j.shared) {
            job_counts(tot, tot32);   // pass1 directly in front
        } else {
            pipe_wait(a.s1_done + j.u, j.chunks, a.status, gave_up, 1, j.u);
            tot = 0; tot32 = 0;
            const int32_t *hb = a.ws_hist + (long long)j.u * kMaxChunks * kBins;
            for (int cc = 0; cc < j.chunks; ++cc) {
                const int v = __ldcg(hb + cc * kBins + lane), v32 = __ldcg(hb + cc * kBins + 32);
                tot += v; tot32 += v32;
                if (cc < j.chunk) { bef += v; bef32 += v32; }
            }
        }
        int T, r, gt_before, eq_before;
        find_threshold(tot, bef, tot32, bef32, pu.keep_rest, lane, T, r, gt_before, eq_before);
        // Per byte b = score + 1 (0 = no token): b + 127 - (T+1) sets bit 7 iff score > T, b + 128 - (T+1) iff
        // score >= T (no byte sum reaches 256); always-kept tokens (kForcedByte) count as S > T for every T.
        const uint32_t T4 = (uint32_t)(T + 1) * 0x01010101u;
        const uint32_t c_gt = 0x7f7f7f7fu - T4, c_ge = 0x80808080u - T4;
        const int written_end = w0 + (w1 - w0 + 255) / 256 * 256;   // pass 1 wrote whole rows (zero bytes past the slice)
        auto flags32 = [&](int first, uint32_t &gt, uint32_t &eq) {      // flags of tokens first .. first + 31
            gt = 0u;
            uint32_t ge = 0u;
            if (first < written_end) {
                const uint4 *p = reinterpret_cast<const uint4 *>(sc + (first - j.t0));
                const uint4 v0 = j.local ? p[0] : __ldcg(p), v1 = j.local ? p[1] : __ldcg(p + 1);
                const uint32_t wv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    gt |= high_bits_to_nibble(wv[e] + c_gt) << (4 * e);
                    ge |= high_bits_to_nibble(wv[e] + c_ge) << (4 * e);
                }
            }
            eq = ge ^ gt;
        };
        // sweep A: how many tokens of this warp's slice lie above / at the threshold
        int mine_gt = 0, mine_eq = 0;
        if (pu.keep > 0) {
            for (int tile = w0; tile < w1; tile += 1024) {
                uint32_t gt, eq;
                flags32(tile + lane * 32, gt, eq);
                mine_gt += __popc(gt);
                mine_eq += __popc(eq);
            }
#pragma unroll
            for (int dd = 16; dd > 0; dd >>= 1) {
                mine_gt += __shfl_xor_sync(0xffffffffu, mine_gt, dd);
                mine_eq += __shfl_xor_sync(0xffffffffu, mine_eq, dd);
            }
        }
        if (lane == 0) { s_wcnt[2 * sw] = mine_gt; s_wcnt[2 * sw + 1] = mine_eq; }
        bar_sync(2, kPipeScoreThreads);
        int32_t *list = a.idx + (long long)pu.b * a.idx_sb + (long long)pu.kvh * a.idx_sh;
        if (pu.keep > 0 && w0 < w1) {
            // tokens before this warp's slice: scored ones of earlier chunks (histograms), always-kept ones before the
            // job (closed form), and everything flagged in the slices of the warps in front
            int run_gt = gt_before + forced_before(pu.wbd, j.t0), run_eq = eq_before;
            for (int w = 0; w < sw; ++w) { run_gt += s_wcnt[2 * w]; run_eq += s_wcnt[2 * w + 1]; }
            // sweep B: the selected tokens at their final positions
            for (int tile = w0; tile < w1; tile += 1024) {              // warp-uniform
                const int first = tile + lane * 32;
                uint32_t gt, eq;
                flags32(first, gt, eq);
                const int packed = __popc(gt) | (__popc(eq) << 16);
                int inc = packed;
#pragma unroll
                for (int dd = 1; dd < 32; dd <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, inc, dd);
                    if (lane >= dd) inc += v;
                }
                const int all = __shfl_sync(0xffffffffu, inc, 31);
                if (packed != 0) {
                    const int excl = inc - packed;
                    int g_run = run_gt + (excl & 0xffff), q_run = run_eq + (int)((unsigned)excl >> 16);
                    write_selected32(list, first, gt, eq, g_run, q_run, r);
                }
                run_gt += all & 0xffff;
                run_eq += (int)((unsigned)all >> 16);
            }
        }
        if (j.chunk == 0) {
            const int st = sw * 32 + lane;
            if (st == 0) a.count[pu.b * a.Hkv + pu.kvh] = pu.keep;
            for (int i = pu.keep + st; i < a.k_max; i += kPipeScoreThreads) list[i] = -1;
        }
        __threadfence();
        bar_sync(2, kPipeScoreThreads);   // also: every warp is done with the score bytes and the counts
        if (sw == 0 && lane == 0) atomicAdd(a.s2_done + j.u, 1);
    }
};

// ------------------------------------------------------------------ the kernel

template <int G>
__global__ void __launch_bounds__(kPipeThreads, 1) pipe_step_kernel(const PipeArgs a) {
    extern __shared__ __align__(128) unsigned char psm[];
    unsigned char *ring = psm;
    float *scratch = reinterpret_cast<float *>(psm + kPipeRingBytes);                       // [8][G][128]
    unsigned char *s_local = psm + kPipeRingBytes + pipe_scratch_bytes(G);
    uint32_t *s_hist = reinterpret_cast<uint32_t *>(s_local + kPipeLocalTokens);
    int *s_pref = reinterpret_cast<int *>(reinterpret_cast<unsigned char *>(s_hist) + kPipeHistBytes);   // [n_units + 1]
    __shared__ int s_cnt[kPipeScoreGroups * kPipeCntStride];
    __shared__ int s_wcnt[2 * kPipeScoreWarps];
    __shared__ float s_m[kPipeGatherWarps][8], s_l[kPipeGatherWarps][8];
    __shared__ uint32_t s_mask[kPipeGatherWarps][kPipeStages];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, P = gridDim.x;
    const int Hq = a.Hq;

    // ---- work split: block counts of all units (from lengths and budgets: nothing here is written by the step)
    for (int v = tid; v < a.n_units; v += kPipeThreads) s_pref[v + 1] = (pipe_unit(a, v).keep + kBlockTokens - 1) / kBlockTokens;
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
    const long long T = s_pref[a.n_units];
    const long long Pe = (T > 0 && T < P) ? T : P;
    const long long x_lo = (T > 0 && cta < Pe) ? (long long)cta * T / Pe : 0;
    const long long x_hi = (T > 0 && cta < Pe) ? (long long)(cta + 1) * T / Pe : 0;
    int u_first = 0;
    {
        int lo = 0, hi = a.n_units;   // largest u with s_pref[u] <= x_lo
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_pref[mid] <= x_lo) lo = mid; else hi = mid;
        }
        u_first = lo;
    }
    pdl_wait();                  // signatures, query signatures, rows: everything older in the stream is final
    pdl_launch_dependents();

    if (warp >= kPipeGatherWarps) {
        // ================================================================ SCORE warps
        const int sw = warp - kPipeGatherWarps;
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPipeScoreRegs));
        ScoreRole<G> S(a, s_local, s_hist, s_cnt, s_wcnt, sw, lane);
        // units without a single selected token take no part in the split: count, padding, zero output
        for (int v = cta; v < a.n_units; v += P) {
            if (s_pref[v + 1] != s_pref[v]) continue;
            const PipeUnit pu = pipe_unit(a, v);
            int32_t *list = a.idx + (long long)pu.b * a.idx_sb + (long long)pu.kvh * a.idx_sh;
            const int st = sw * 32 + lane;
            for (int i = st; i < a.k_max; i += kPipeScoreThreads) list[i] = -1;
            const long long h0 = (long long)pu.b * Hq + (long long)pu.kvh * G;
            for (int i = st; i < G * kD; i += kPipeScoreThreads) a.out[h0 * kD + i] = 0;
            if (st == 0) a.count[v] = 0;
            if (a.lse && st < G) a.lse[h0 + st] = -CUDART_INF_F;
        }
        if (x_lo >= x_hi) return;
        // the units of this CTA's range; the first and the last may be shared with neighbours
        auto job_of = [&](int u, ScoreJob &j, PipeUnit &pu, bool single) -> bool {   // false: this CTA scores nothing of u
            pu = pipe_unit(a, u);
            const PipeSplit sp = pipe_split(s_pref[u], s_pref[u + 1], T, Pe);
            j.u = u;
            if (sp.n_parts == 1) {
                j.chunk = 0; j.chunks = 1; j.t0 = 0; j.t1 = pu.n; j.shared = false;
                j.local = pu.n <= kPipeLocalTokens;
                return true;
            }
            j.shared = true;
            j.chunks = pipe_chunks(pu.n, sp.n_parts);
            j.chunk = cta - sp.c_first;
            if (j.chunk >= j.chunks) return false;
            const int ct = pipe_chunk_tokens(pu.n, j.chunks);
            j.t0 = min(pu.n, j.chunk * ct);
            j.t1 = min(pu.n, j.t0 + ct);
            j.local = single && (j.t1 - j.t0) <= kPipeLocalTokens;
            return true;
        };
        int u_last = u_first;
        for (int u = u_first; u < a.n_units && s_pref[u] < x_hi; ++u)
            if (s_pref[u + 1] > s_pref[u]) u_last = u;
        while (s_pref[u_first + 1] == s_pref[u_first]) ++u_first;
        const bool first_shared = pipe_split(s_pref[u_first], s_pref[u_first + 1], T, Pe).n_parts > 1;
        const bool last_shared = u_last != u_first && pipe_split(s_pref[u_last], s_pref[u_last + 1], T, Pe).n_parts > 1;
        const bool single = (u_first == u_last);
        ScoreJob jf, jl;
        PipeUnit pf, pl;
        bool have_f = false, have_l = false;
        // 1. first passes of the shared units, so that no neighbour waits for this CTA's whole range
        if (first_shared) {
            have_f = job_of(u_first, jf, pf, single);
            if (have_f) { S.pass1(jf, pf); S.publish_chunk(jf); }
        }
        if (last_shared) {
            have_l = job_of(u_last, jl, pl, false);
            if (have_l) { S.pass1(jl, pl); S.publish_chunk(jl); }
        }
        // 2. their second passes: the GATHER warps here need the first unit's list first, and a neighbour's need the last
        // unit's (it is the first of its range)
        if (have_f) S.pass2(jf, pf);
        if (have_l) S.pass2(jl, pl);
        // 3. the units inside the range, in order
        for (int u = u_first + (first_shared ? 1 : 0); u <= u_last - (last_shared ? 1 : 0); ++u) {
            if (s_pref[u + 1] == s_pref[u]) continue;
            ScoreJob j;
            PipeUnit pu;
            job_of(u, j, pu, false);
            S.pass1(j, pu);
            S.pass2(j, pu);
        }
        return;
    }

    // ==================================================================== GATHER warps
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPipeGatherRegs));
    if (x_lo >= x_hi) return;
    const int g = lane >> 2, c = lane & 3;
    unsigned char *my_ring = ring + warp * kPipeWarpRing;
    const uint32_t ring_u32 = smem_u32(my_ring);
    const bool paged = a.block_table != nullptr;
    const long long k_row = a.K.sn * 2, v_row = a.V.sn * 2;
    bool gave_up = false;

    // a segment = the blocks of one unit inside this CTA's range
    struct Seg {
        int u, blk_lo, blk_hi;     // blocks of the unit (16 entries each)
        int n_parts, my_part, slot0;
        long long x_next;          // where the next segment starts in the global block sequence
    };
    auto seg_at = [&](long long x, int u) -> Seg {
        Seg s;
        s.u = u;
        const long long u_lo = s_pref[u], u_hi = s_pref[u + 1];
        const PipeSplit sp = pipe_split(u_lo, u_hi, T, Pe);
        s.n_parts = sp.n_parts;
        s.my_part = cta - sp.c_first;
        s.slot0 = sp.c_first + u;
        const long long e = (x_hi < u_hi) ? x_hi : u_hi;
        s.blk_lo = (int)(x - u_lo);
        s.blk_hi = (int)(e - u_lo);
        s.x_next = e;
        return s;
    };
    auto next_unit = [&](int u) { ++u; while (u < a.n_units && s_pref[u + 1] == s_pref[u]) ++u; return u; };
    // Has every chunk of unit u been through its second pass?  A warp asks from both of its cursors, and the counter of
    // a unit goes back to zero once the unit is finished (which needs this warp's consume side, but not its issue side,
    // to have seen it): what was seen once is remembered.  Units are visited in ascending order by both cursors.
    int known_ready = -1;
    auto unit_ready = [&](int u, int n, int n_parts) -> bool {
        if (u <= known_ready || gave_up) return true;
        const int want = (n_parts == 1) ? 1 : pipe_chunks(n, n_parts);
        if (ld_acquire(a.s2_done + u) < want) return false;
        known_ready = u;
        return true;
    };

    // ---- issue side: the next block whose rows are to be requested
    int i_u = u_first;
    while (s_pref[i_u + 1] == s_pref[i_u]) ++i_u;
    long long i_x = x_lo;
    bool i_setup = false, i_have = false;   // segment parameters valid / list entry of the next block prefetched
    int i_blk = 0, i_blk_hi = 0, i_n = 0, i_keep = 0, i_raw = -1;
    long long i_xnext = 0;
    const int32_t *i_list = nullptr, *i_pages = nullptr;
    const unsigned char *i_Kb = nullptr, *i_Vb = nullptr;
    // Makes (segment, block) point at the next block of this warp with its list entry on the way; false: the
    // unit is not released yet, or the range is exhausted.
    auto issue_prepare = [&]() -> bool {
        while (true) {
            if (i_x >= x_hi) return false;
            if (!i_setup) {
                const PipeUnit pu = pipe_unit(a, i_u);
                const Seg s = seg_at(i_x, i_u);
                if (!unit_ready(i_u, pu.n, s.n_parts)) return false;
                i_n = pu.n; i_keep = pu.keep;
                i_blk = s.blk_lo + warp; i_blk_hi = s.blk_hi; i_xnext = s.x_next;
                i_list = a.idx + (long long)pu.b * a.idx_sb + (long long)pu.kvh * a.idx_sh;
                i_Kb = reinterpret_cast<const unsigned char *>(a.K.ptr + (paged ? 0LL : (long long)pu.b * a.K.sb) + (long long)pu.kvh * a.K.sh);
                i_Vb = reinterpret_cast<const unsigned char *>(a.V.ptr + (paged ? 0LL : (long long)pu.b * a.V.sb) + (long long)pu.kvh * a.V.sh);
                i_pages = paged ? a.block_table + (long long)pu.b * a.bt_sb : nullptr;
                i_setup = true;
            }
            if (i_blk < i_blk_hi) {
                const int p = i_blk * kBlockTokens + (lane & 15);
                i_raw = (p < i_keep) ? __ldcg(i_list + p) : -1;
                return true;
            }
            i_x = i_xnext;
            i_u = next_unit(i_u);
            i_setup = false;
        }
    };
    auto issue_block = [&](int stg) {
        int t = i_raw;
        if (t >= i_n) t = -1;   // cannot happen with lists written by this kernel; keeps a given-up run inside the cache
        if (paged && t >= 0) t = __ldg(i_pages + (t >> a.page_shift)) * a.page_rows + (t & ((1 << a.page_shift) - 1));
        const uint32_t valid = attn_issue_block(ring_u32 + stg * kStageBytes, i_Kb, i_Vb, k_row, v_row, t, lane);
        if (lane == 0) s_mask[warp][stg] = valid;
        i_blk += kPipeGatherWarps;
    };

    // ---- consume side
    int c_u = i_u;
    long long c_x = x_lo;
    bool c_setup = false;
    Seg cs{};
    int c_left = 0;            // blocks of this warp still to consume in the segment
    long long head0 = 0;
    uint32_t qa[8][2];
    float acc[8][4];
    float m_run = -CUDART_INF_F, l_run = 0.0f;
    int inflight = 0, st_issue = 0, st_cons = 0, idle = 0;

    while (true) {
        // top up the ring
        while (inflight < kPipeStages) {
            if (!i_have) { i_have = issue_prepare(); if (!i_have) break; }
            issue_block(st_issue);
            cp_async_commit();
            st_issue ^= 1;
            ++inflight;
            i_have = issue_prepare();   // the next entry travels while rows are consumed
            if (!i_have) break;
        }
        if (c_x >= x_hi) break;
        if (!c_setup) {
            const PipeUnit pu = pipe_unit(a, c_u);
            cs = seg_at(c_x, c_u);
            if (!unit_ready(c_u, pu.n, cs.n_parts)) {   // only a segment without blocks for this warp gets here unreleased
                if (++idle > kPipeSpinLimit) { gave_up = true; pipe_give_up(a.status, 2, c_u, cs.n_parts, ld_acquire(a.s2_done + c_u)); }
                if ((idle & 63) == 0 && ld_acquire(reinterpret_cast<const int32_t *>(a.status + 1)) != 0) gave_up = true;
                __nanosleep(200);
                continue;
            }
            head0 = (long long)pu.b * Hq + (long long)pu.kvh * G;
            attn_load_q<G>(qa, a.q + head0 * kD, lane);
#pragma unroll
            for (int mt = 0; mt < 8; ++mt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
            m_run = -CUDART_INF_F; l_run = 0.0f;
            const int first = cs.blk_lo + warp;
            c_left = (first < cs.blk_hi) ? (cs.blk_hi - first + kPipeGatherWarps - 1) / kPipeGatherWarps : 0;
            c_setup = true;
        }
        if (c_left > 0) {
            if (inflight == 0) {   // the issue side is waiting for the unit's release
                if (++idle > kPipeSpinLimit) { gave_up = true; pipe_give_up(a.status, 3, i_u, (int)i_x, ld_acquire(a.s2_done + min(i_u, a.n_units - 1))); }
                if ((idle & 63) == 0 && ld_acquire(reinterpret_cast<const int32_t *>(a.status + 1)) != 0) gave_up = true;
                __nanosleep(200);
                continue;
            }
            if (inflight == 2) cp_async_wait<1>(); else cp_async_wait<0>();
            __syncwarp();
            const uint32_t ks = ring_u32 + st_cons * kStageBytes;
            attn_consume_block(ks, ks + kTileBytes, s_mask[warp][st_cons], qa, a.scale_log2, lane, acc, m_run, l_run);
            __syncwarp();
            st_cons ^= 1;
            --inflight;
            --c_left;
            idle = 0;
            if (c_left > 0) continue;
        }
        // ---- the segment is done for this warp: merge the eight warps, then publish or finish the unit
        {
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            if (c == 0) { s_m[warp][g] = m_run; s_l[warp][g] = l_run; }
            float *my_acc = scratch + warp * G * kD;
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
            bar_sync(1, kPipeGatherThreads);
            const int d = tid & (kD - 1), hsel = tid >> 7;
            const bool split = cs.n_parts > 1;
            float Mj[(G + 1) / 2], Lj[(G + 1) / 2], Aj[(G + 1) / 2];   // this thread's heads: hsel, hsel + 2, ...
#pragma unroll
            for (int jj = 0; jj < (G + 1) / 2; ++jj) {
                const int j = (G == 1) ? 0 : 2 * jj + hsel;
                float M = s_m[0][j];
#pragma unroll
                for (int w = 1; w < kPipeGatherWarps; ++w) M = fmaxf(M, s_m[w][j]);
                float L = 0.0f, A = 0.0f;
                if (M > -CUDART_INF_F) {
#pragma unroll
                    for (int w = 0; w < kPipeGatherWarps; ++w) {
                        const float f = exp2f(s_m[w][j] - M);
                        L = fmaf(s_l[w][j], f, L);
                        A = fmaf(scratch[(w * G + j) * kD + d], f, A);
                    }
                }
                Mj[jj] = M; Lj[jj] = L; Aj[jj] = A;
            }
            const bool mine = (G > 1) || hsel == 0;   // with one head per group the second half of the threads idles
            bool finalize = !split;
            if (split) {
                const long long slot = (long long)(cs.slot0 + cs.my_part) * G;
                if (mine) {
#pragma unroll
                    for (int jj = 0; jj < (G + 1) / 2; ++jj) {
                        const int j = (G == 1) ? 0 : 2 * jj + hsel;
                        a.part_acc[(slot + j) * kD + d] = Aj[jj];
                        if (d == 0) { a.part_ml[(slot + j) * 2] = Mj[jj]; a.part_ml[(slot + j) * 2 + 1] = Lj[jj]; }
                    }
                }
                __threadfence();
                bar_sync(1, kPipeGatherThreads);
                if (tid == 0) {
                    const int t = atomicAdd(&a.tickets[cs.u], 1);
                    s_last = (t == cs.n_parts - 1);
                    if (s_last) a.tickets[cs.u] = 0;   // ready for the next call
                }
                bar_sync(1, kPipeGatherThreads);
                finalize = (s_last != 0);
                if (finalize) {
                    __threadfence();
                    // merge of the parts: thread (d, hsel) folds its heads over all parts, a few loads in flight at a time
#pragma unroll
                    for (int jj = 0; jj < (G + 1) / 2; ++jj) {
                        const int j = (G == 1) ? 0 : 2 * jj + hsel;
                        float M = -CUDART_INF_F, L = 0.0f, A = 0.0f;
                        if (mine) {
                            for (int p0 = 0; p0 < cs.n_parts; p0 += 8) {
                                float av[8], mv[8], lv[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const bool ok = p0 + e < cs.n_parts;
                                    const long long sl = (long long)(cs.slot0 + (ok ? p0 + e : 0)) * G + j;
                                    const float2 ml = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + sl * 2));
                                    av[e] = __ldcg(a.part_acc + sl * kD + d);
                                    mv[e] = ok ? ml.x : -CUDART_INF_F;
                                    lv[e] = ok ? ml.y : 0.0f;
                                }
                                float Mn = M;
#pragma unroll
                                for (int e = 0; e < 8; ++e) Mn = fmaxf(Mn, mv[e]);
                                if (Mn > -CUDART_INF_F) {
                                    const float f0 = exp2f(M - Mn);
                                    L *= f0; A *= f0;
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        const float f = exp2f(mv[e] - Mn);   // 0 for absent parts
                                        L = fmaf(lv[e], f, L);
                                        A = fmaf(av[e], f, A);
                                    }
                                    M = Mn;
                                }
                            }
                        }
                        Mj[jj] = M; Lj[jj] = L; Aj[jj] = A;
                    }
                }
            }
            if (finalize) {
                if (mine) {
#pragma unroll
                    for (int jj = 0; jj < (G + 1) / 2; ++jj) {
                        const int j = (G == 1) ? 0 : 2 * jj + hsel;
                        const float o = (Lj[jj] > 0.0f) ? Aj[jj] / Lj[jj] : 0.0f;
                        const __nv_bfloat16 ob = __float2bfloat16_rn(o);
                        a.out[(head0 + j) * kD + d] = *reinterpret_cast<const uint16_t *>(&ob);
                        if (a.lse && d == 0) a.lse[head0 + j] = (Lj[jj] > 0.0f) ? (Mj[jj] * kLn2 + logf(Lj[jj])) : -CUDART_INF_F;
                    }
                }
                // every part of the unit has seen its release: the counters go back to zero for the next call
                if (tid == 0) { a.s1_done[cs.u] = 0; a.s2_done[cs.u] = 0; }
            }
            bar_sync(1, kPipeGatherThreads);   // the scratch and s_m / s_l are free again
        }
        c_x = cs.x_next;
        c_u = next_unit(c_u);
        c_setup = false;
    }
    cp_async_wait<0>();
}

// ------------------------------------------------------------------ host side

template <int G>
static int pipe_prepare() {   // opt in to the shared memory once per device; returns resident CTAs per SM (0 on error)
    static int per_sm[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!per_sm[dev]) {
        if (cudaFuncSetAttribute(pipe_step_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, pipe_smem_bytes(G)) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pipe_step_kernel<G>, kPipeThreads, pipe_smem_bytes(G)) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            return 0;
        }
        per_sm[dev] = n;
    }
    return per_sm[dev];
}

// The pipelined kernel serves steps of more units than the single-cluster kernel holds, up to kMaxBalancedUnits.
bool pipe_step_eligible(int B, int Hq, int Hkv) {
    if (Hkv <= 0 || (long long)B * Hkv > kMaxBalancedUnits) return false;
    switch (Hq / Hkv) {
        case 1: return pipe_prepare<1>() > 0;
        case 2: return pipe_prepare<2>() > 0;
        case 4: return pipe_prepare<4>() > 0;
        case 8: return pipe_prepare<8>() > 0;
        default: return false;
    }
}

template <int G>
static cudaError_t launch_pipe_g(const PipeArgs &args, cudaStream_t st) {
    if (pipe_prepare<G>() <= 0) return cudaErrorInvalidConfiguration;
    // one CTA per SM: all of them resident at once, whatever the batch
    cudaError_t e = launch_pdl(pipe_step_kernel<G>, dim3(sm_count()), dim3(kPipeThreads), (size_t)pipe_smem_bytes(G), st, args);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_pipe_step(int B, int Hq, int Hkv, float sm_scale, const uint32_t *q_codes, const uint32_t *k_codes,
                             long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq, int k_uniform,
                             int max_seq_len, int k_max, int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                             const uint16_t *q, TensorView K, TensorView V, uint16_t *out, float *lse, int32_t *tickets,
                             int32_t *s1_done, int32_t *s2_done, int32_t *ws_hist, unsigned char *ws_scores, long long score_row,
                             float *part_ml, float *part_acc, uint32_t *status, cudaStream_t st, Windows win,
                             const int32_t *block_table, long long bt_sb, int page_shift) {
    PipeArgs a{};
    a.q_codes = q_codes; a.k_codes = k_codes; a.kc_sb = kc_sb; a.kc_sh = kc_sh; a.seq_lens = seq_lens; a.k_per_seq = k_per_seq;
    a.k_uniform = k_uniform; a.max_seq_len = max_seq_len; a.k_max = k_max; a.win = win; a.idx = idx; a.idx_sb = idx_sb;
    a.idx_sh = idx_sh; a.count = count; a.q = q; a.K = K; a.V = V; a.block_table = block_table; a.bt_sb = bt_sb;
    a.page_shift = page_shift; a.page_rows = (block_table && K.sn > 0) ? (int)(K.sb / K.sn) : 0;
    a.scale_log2 = sm_scale * kLog2e; a.out = out; a.lse = lse; a.Hq = Hq; a.Hkv = Hkv; a.n_units = B * Hkv;
    a.tickets = tickets; a.s1_done = s1_done; a.s2_done = s2_done; a.ws_hist = ws_hist; a.ws_scores = ws_scores;
    a.score_row = score_row; a.part_ml = part_ml; a.part_acc = part_acc; a.status = status;
    switch (Hq / Hkv) {
        case 1: return launch_pipe_g<1>(a, st);
        case 2: return launch_pipe_g<2>(a, st);
        case 4: return launch_pipe_g<4>(a, st);
        case 8: return launch_pipe_g<8>(a, st);
        default: return cudaErrorInvalidValue;
    }
}

} // namespace ha
