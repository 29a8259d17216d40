// Device-side building blocks of the SCORE + TOPK kernels (included by ha_score_topk.cu and ha_fused.cu).
#pragma once

#include "ha_common.cuh"

namespace ha {

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

// The same two helpers over a paged signature cache (pool_head = pool + h * head_stride, table_b = the sequence's row of
// the block table).  Pages of at least four tokens hold an aligned group of four in one piece; smaller pages are read
// token by token.
__device__ __forceinline__ uint4 load_codes4_paged(const CodePages &cp, const uint32_t *pool_head, const int32_t *table_b,
                                                   int base, int n) {
    if (cp.shift >= 2) {
        const uint32_t *p = pool_head + (long long)__ldg(table_b + (base >> cp.shift)) * cp.page_stride + (base & ((1 << cp.shift) - 1));
        return load_codes4(p - base, base, n);
    }
    uint32_t v[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = base + i;
        if (t < n) v[i] = __ldg(pool_head + (long long)__ldg(table_b + (t >> cp.shift)) * cp.page_stride + (t & ((1 << cp.shift) - 1)));
    }
    return make_uint4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void patch_token_paged(uint4 &v, int base, int last, const CodePages &cp, const uint32_t *pool_head,
                                                  const int32_t *table_b) {
    const int e = last - base;
    if (e < 0 || e > 3) return;
    const uint32_t c = __ldcg(pool_head + (long long)__ldg(table_b + (last >> cp.shift)) * cp.page_stride + (last & ((1 << cp.shift) - 1)));
    if (e == 0) v.x = c; else if (e == 1) v.y = c; else if (e == 2) v.z = c; else v.w = c;
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


// Score byte of a token that is always in context (Windows): above every real score + 1 (<= 33), so the
// flag arithmetic below sees "score > T" for every threshold, and small enough that no byte sum reaches 256.
constexpr uint32_t kForcedByte = 63u;

// Bits 7, 15, 23, 31 of x gathered into a nibble (bit e = bit 7 of byte e).  The four partial products
// land on distinct bit positions, so the multiplication carries nothing into bits 28..31.
__device__ __forceinline__ uint32_t high_bits_to_nibble(uint32_t x) {
    return ((x & 0x80808080u) * 0x00204081u) >> 28;
}

// Index of the single set bit of `one_hot`.
__device__ __forceinline__ int one_hot_index(uint32_t one_hot) {
    return ((one_hot & 0xaaaaaaaau) ? 1 : 0) | ((one_hot & 0xccccccccu) ? 2 : 0) | ((one_hot & 0xf0f0f0f0u) ? 4 : 0) |
           ((one_hot & 0xff00ff00u) ? 8 : 0) | ((one_hot & 0xffff0000u) ? 16 : 0);
}

// Visits the flagged tokens among 32 consecutive tokens from `first` on in ascending order; g_run / q_run
// count the tokens with S > T / S == T seen so far in the whole sequence; r tokens of score T are wanted.
// sink(position in the index list, token) is called for every selected token.
template <typename Sink>
__device__ __forceinline__ void visit_selected32(int first, uint32_t gt, uint32_t eq, int &g_run, int &q_run, int r,
                                                 Sink &&sink) {
    uint32_t m = gt | eq;
    while (m) {
        const uint32_t lb = m & (0u - m);
        m ^= lb;
        const int t = first + one_hot_index(lb);
        if (gt & lb) { sink(g_run + min(q_run, r), t); ++g_run; }
        else { if (q_run < r) sink(g_run + q_run, t); ++q_run; }
    }
}
__device__ __forceinline__ void write_selected32(int32_t *list, int first, uint32_t gt, uint32_t eq, int &g_run,
                                                 int &q_run, int r) {
    visit_selected32(first, gt, eq, g_run, q_run, r, [&](int pos, int t) { list[pos] = t; });
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
