// Device-side building blocks of the SCORE + TOPK kernels (included by ha_score_topk.cu and ha_fused.cu).
#pragma once

#include "ha_common.cuh"

namespace ha {

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

// Re-read token `last` (coherently) if it lies in [base, base+4): it may have been written by the
// kernel this one was launched behind.
__device__ __forceinline__ void patch_token(uint4 &v, int base, int last, const uint32_t *row) {
    const int e = last - base;
    if (e < 0 || e > 3) return;
    const uint32_t c = __ldcg(row + last);
    if (e == 0) v.x = c; else if (e == 1) v.y = c; else if (e == 2) v.z = c; else v.w = c;
}

// Four group scores packed as bytes holding score + 1 (1..33); a zero byte means "no token".
template <int G>
__device__ __forceinline__ uint32_t scores4(const uint4 &c, const uint32_t (&qc)[G]) {
    return (uint32_t)(group_score<G>(c.x, qc) + 1) | ((uint32_t)(group_score<G>(c.y, qc) + 1) << 8) |
           ((uint32_t)(group_score<G>(c.z, qc) + 1) << 16) | ((uint32_t)(group_score<G>(c.w, qc) + 1) << 24);
}

// Per-byte flags (bit 7 of each byte) of "score > T" and "score == T" for four packed score+1 bytes.
// Plain 32-bit arithmetic: with bytes <= 33 and T + 1 <= 34 no byte sum reaches 256, so no carry
// crosses a byte; a zero byte (no token) is neither above nor equal to any threshold.
__device__ __forceinline__ void flags4(uint32_t s4, uint32_t t1x4, uint32_t &gt, uint32_t &eq) {
    gt = (s4 + (0x7f7f7f7fu - t1x4)) & 0x80808080u;            // byte + 127 - (T+1) >= 128  <=>  score > T
    const uint32_t ge = (s4 + (0x80808080u - t1x4)) & 0x80808080u;   // byte + 128 - (T+1) >= 128  <=>  score >= T
    eq = ge ^ gt;
}

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// read an int of CTA `rank`'s shared memory at the address that `local` has in this CTA
__device__ __forceinline__ int ld_dsmem(const int *local, uint32_t rank) {
    uint32_t a = (uint32_t)__cvta_generic_to_shared(local), ra;
    int v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(ra) : "memory");
    return v;
}


// The four bit-7 flags of a word gathered into a nibble (bit e = flag of byte e).
__device__ __forceinline__ uint32_t flags_to_nibble(uint32_t f) {
    return ((((f >> 7) & 0x01010101u) * 0x01020408u) >> 24) & 0xfu;
}

// Writes the selected tokens among 16 consecutive tokens starting at `first`: gt16 / eq16 are the
// per-token flags "score > T" / "score == T" (bit e = token first + e); gt_lt / eq_lt count the
// tokens before `first` with those properties; r tokens of score T are still wanted overall.
// Only the flagged tokens are visited; each position comes from popcounts, not from a running sum.
__device__ __forceinline__ void write_selected16(int32_t *list, int first, uint32_t gt16, uint32_t eq16, int gt_lt,
                                                 int eq_lt, int r) {
    uint32_t m = gt16 | eq16;
    while (m) {
        const int e = __ffs((int)m) - 1;
        m &= m - 1;
        const uint32_t below = (1u << e) - 1u;
        const int g = gt_lt + __popc(gt16 & below), q = eq_lt + __popc(eq16 & below);
        if ((gt16 >> e) & 1u) list[g + min(q, r)] = first + e;
        else if (q < r) list[g + q] = first + e;
    }
}

// Warp-wide threshold search over the 33 score levels.  Lane l passes the count of level l (tot) and
// the part of it that lies before the caller's own slice (bef); level 32 comes in tot32 / bef32.
// Returns T = largest level with #{S >= T} >= keep, r = keep - #{S > T}, and the numbers of tokens
// before the caller's slice with S > T and with S == T.  keep == 0 gives T = 33 (nothing selected).
__device__ __forceinline__ void find_threshold(int tot, int bef, int tot32, int bef32, int keep, int lane, int &T,
                                               int &r, int &gt_before, int &eq_before) {
    int st = tot, sb = bef;   // suffix sums over levels lane..31
#pragma unroll
    for (int dd = 1; dd < 32; dd <<= 1) {
        const int vt = __shfl_down_sync(0xffffffffu, st, dd), vb = __shfl_down_sync(0xffffffffu, sb, dd);
        if (lane + dd < 32) { st += vt; sb += vb; }
    }
    st += tot32;   // #{S >= lane}
    sb += bef32;   // same, restricted to what lies before the caller's slice
    T = kBins; r = 0; gt_before = 0; eq_before = 0;
    if (keep > 0) {
        const unsigned ge = __ballot_sync(0xffffffffu, st >= keep);
        if (tot32 >= keep) { T = 32; r = keep; gt_before = 0; eq_before = bef32; }
        else {
            T = 31 - __clz(ge);   // ge != 0 because #{S >= 0} = n >= keep
            const int above = __shfl_sync(0xffffffffu, st, min(T + 1, 31));      // #{S >= T+1}
            const int above_b = __shfl_sync(0xffffffffu, sb, min(T + 1, 31));
            const int at_b = __shfl_sync(0xffffffffu, bef, T);
            const int gt = (T == 31) ? tot32 : above;
            r = keep - gt;
            gt_before = (T == 31) ? bef32 : above_b;
            eq_before = at_b;
        }
    }
}

} // namespace ha
