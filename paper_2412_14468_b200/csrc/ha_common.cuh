// Internal declarations shared by the translation units of libhashattn (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hashattn.h"

namespace ha {

constexpr int kD = HA_HEAD_DIM;     // head dimension, mapping input width
constexpr int kHid = 128;           // mapping hidden width
constexpr int kBits = HA_N_BITS;    // signature width b
constexpr int kBins = HA_HIST_BINS; // score levels 0..32
constexpr int kMaxChunks = 128;     // chunks of the code scan per (sequence, KV head)
constexpr int kMaxAttnCtas = 1024;  // persistent CTAs of the attention kernel (bounds the partial slots)
constexpr int kMaxBalancedUnits = 1024;   // above this many (sequence, KV head) units: one CTA per unit
constexpr int kMaxGroup = 8;        // query heads per KV head
constexpr size_t kHeaderBytes = 256;   // device status word (+ padding)
constexpr int kMaxUnits = 65536;       // (sequence, KV head) pairs: bounds the ticket region

// Where each scratch region lives inside the caller's workspace.  All regions but the last depend
// on the head counts and the batch only; the score bytes of the long-sequence scan come last and
// grow with the maximum sequence length, so a workspace sized once serves every smaller call.
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct WorkspaceLayout {
    size_t off_tickets;   // i32 [3][B][Hkv]  arrival counters of the split-K merge, then the two release counters per unit
                          // of the pipelined step (first pass / second pass of SCORE + TOPK done); all zero between calls
    size_t off_hist;      // i32 [B][Hkv][kMaxChunks][33]   per-chunk score histograms
    size_t off_part_ml;   // f32 [slots][G][2]    split-K running max (log2 domain) and sum, slots = kMaxAttnCtas + B*Hkv
    size_t off_part_acc;  // f32 [slots][G][128]  split-K unnormalised outputs
    size_t off_stage_q;   // bf16 [B][Hq][128]              host-entry staging
    size_t off_stage_k;   // bf16 [B][Hkv][128]
    size_t off_stage_v;   // bf16 [B][Hkv][128]
    size_t off_stage_out; // bf16 [B][Hq][128]
    size_t off_qcodes;    // u32 [B][Hq]
    size_t off_scores;    // u8 [B][Hkv][round_up(max_seq_len, 256)]  group scores (long-sequence path, shared units of the pipelined step)
    size_t total;
};

inline size_t score_row_bytes(int max_seq_len) { return align_up((size_t)(max_seq_len > 0 ? max_seq_len : 0), 256); }

inline WorkspaceLayout make_layout(int B, int Hq, int Hkv, int max_seq_len) {
    WorkspaceLayout L;
    size_t o = kHeaderBytes;
    L.off_tickets = o;   o = align_up(o + (size_t)3 * B * Hkv * 4, 256);
    L.off_hist = o;      o = align_up(o + (size_t)B * Hkv * kMaxChunks * kBins * 4, 256);
    const size_t slots = (size_t)kMaxAttnCtas + (size_t)B * Hkv, G = (size_t)(Hq / (Hkv > 0 ? Hkv : 1));
    L.off_part_ml = o;   o = align_up(o + slots * G * 2 * 4, 256);
    L.off_part_acc = o;  o = align_up(o + slots * G * kD * 4, 256);
    L.off_stage_q = o;   o = align_up(o + (size_t)B * Hq * kD * 2, 256);
    L.off_stage_k = o;   o = align_up(o + (size_t)B * Hkv * kD * 2, 256);
    L.off_stage_v = o;   o = align_up(o + (size_t)B * Hkv * kD * 2, 256);
    L.off_stage_out = o; o = align_up(o + (size_t)B * Hq * kD * 2, 256);
    L.off_qcodes = o;    o = align_up(o + (size_t)B * Hq * 4, 256);
    L.off_scores = o;    o = align_up(o + (size_t)B * Hkv * score_row_bytes(max_seq_len), 256);
    L.total = o;
    return L;
}

// Tokens of the code cache scanned by one CTA of the long-sequence path: the sequence is cut into equal
// chunks (a multiple of 16 tokens, at least one pass of 256 threads x 16 tokens) so that the grid has
// about three and a half CTAs per SM when there is that much work (four stay resident of either kernel;
// filling every slot made the whole step slower, because the CTAs of the kernel behind could not become
// resident early), and so that a sequence of max_seq_len tokens needs at most kMaxChunks chunks.
inline int chunk_tokens_for(int n_units, int max_seq_len, int n_sm) {
    const long long units = n_units > 0 ? n_units : 1, n = max_seq_len > 0 ? max_seq_len : 1;
    long long per_unit = 7LL * (n_sm > 0 ? n_sm : 148) / 2 / units;
    if (per_unit < 1) per_unit = 1;
    if (per_unit > kMaxChunks) per_unit = kMaxChunks;
    long long c = (n + per_unit - 1) / per_unit;
    if (c < 4096) c = 4096;
    const long long c_min = (n + kMaxChunks - 1) / kMaxChunks;
    if (c < c_min) c = c_min;
    return (int)((c + 15) / 16 * 16);
}

// ---- programmatic dependent launch: a kernel launched with launch_pdl may start while its
// predecessor in the stream is still running; everything it reads from, or writes over, earlier
// work must come after pdl_wait().
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

void count_launch(int n = 1);

struct TensorView {
    const uint16_t *ptr;
    long long sb, sh, sn;
};

struct MapView {
    const uint16_t *w1, *w2, *w3;
    const float *b1, *b2, *b3;
};

// Tokens that are always in context (Section 5, paragraph on baselines): the first n_sink and the most
// recent n_local of a sequence; the budget k counts the heavy tokens retrieved in addition.
struct Windows {
    int n_sink, n_local;
};
// For a sequence of n tokens: token t is forced iff t < sink_end or t >= local_begin.
struct WindowBounds {
    int sink_end, local_begin;   // sink_end <= local_begin <= n (touching or overlapping windows: equal)
};
#ifdef __CUDACC__
__host__ __device__
#endif
inline WindowBounds window_bounds(Windows w, int n) {
    WindowBounds r;
    r.sink_end = w.n_sink < n ? w.n_sink : n;
    const int lb = n - w.n_local;
    r.local_begin = lb > r.sink_end ? lb : r.sink_end;
    return r;
}
// number of forced tokens with index < p (0 <= p <= n)
#ifdef __CUDACC__
__host__ __device__
#endif
inline int forced_before(WindowBounds w, int p) {
    return (p < w.sink_end ? p : w.sink_end) + (p > w.local_begin ? p - w.local_begin : 0);
}

// A paged signature cache (the paper's vLLM integration keeps the KV cache, and with it the signatures of Section 4.1,
// in pages addressed through a block table): token t of sequence b and KV head h is the 32-bit word
// pool[table[b * bt_sb + (t >> shift)] * page_stride + h * head_stride + (t & (2^shift - 1))].  table == NULL: contiguous.
struct CodePages {
    const int32_t *table;
    long long bt_sb, page_stride, head_stride;
    int shift;
};

// One batch of single vectors to encode (decode step): CTA i handles sequence i / n_nets and
// network i % n_nets, i.e. the heads_per_kv (<= 8) heads that share that network.
struct EncodeJob {
    const uint16_t *x;       // bf16, vector (b,h) at x + b*x_sb + h*x_sh
    long long x_sb, x_sh;
    uint32_t *codes;         // written at codes + b*c_sb + h*c_sh + slot
    long long c_sb, c_sh;
    const int32_t *slot;     // per-sequence slot (device) or NULL = 0
    int slot_minus_one;      // 1: slot[] holds sequence lengths, write at slot[b] - 1
    int n_heads, heads_per_kv, n_cta;   // n_cta = batch * n_heads / heads_per_kv
    int batch, cta_per_net;  // filled in by the launcher: sequences, and CTAs that share one network's items
    MapView map;
    CodePages pages;         // pages.table != NULL: `codes` is a paged pool and the slot a token of the sequence
};
#ifdef __CUDACC__
// where the signature of (sequence b, head h, token slot) is stored
__device__ __forceinline__ uint32_t *encode_slot_ptr(const EncodeJob &J, int b, int h, int slot) {
    if (J.pages.table)
        return J.codes + (long long)J.pages.table[(long long)b * J.pages.bt_sb + (slot >> J.pages.shift)] * J.pages.page_stride +
               (long long)h * J.pages.head_stride + (slot & ((1 << J.pages.shift) - 1));
    return J.codes + (long long)b * J.c_sb + (long long)h * J.c_sh + slot;
}
#endif

// Number of SMs of the current device (cached per device).
inline int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// ---- launchers (each enqueues kernels on `st` and returns the last CUDA error) ----
cudaError_t launch_encode_vectors(const EncodeJob &a, const EncodeJob &b, cudaStream_t st);
cudaError_t launch_encode_bulk(const MapView &map, int heads_per_kv, TensorView x, int B, int H, int T,
                               uint32_t *codes, long long c_sb, long long c_sh, cudaStream_t st);
cudaError_t launch_encode_tc(const MapView &map, int heads_per_kv, TensorView x, int B, int H, int T, uint32_t *codes,
                             long long c_sb, long long c_sh, cudaStream_t st);
cudaError_t launch_encode_umma(const MapView &map, int heads_per_kv, TensorView x, int B, int H, int T, uint32_t *codes,
                               long long c_sb, long long c_sh, uint32_t *status, cudaStream_t st);

cudaError_t launch_score_topk(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes,
                              long long kc_sb, long long kc_sh, const int32_t *seq_lens,
                              const int32_t *k_per_seq, int k_uniform, int max_seq_len, int k_max,
                              int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                              int32_t *hist_out, int32_t *ws_hist, unsigned char *ws_scores, cudaStream_t st, Windows win = Windows{0, 0},
                              CodePages pages = CodePages{nullptr, 0, 0, 0, 0}, int row_shift = -1);
// pages.table != NULL: k_codes is a paged pool (always the two-kernel path); row_shift >= 0: one unit per QUERY head
// (Hq units per sequence, groups of one head), whose signature row is that of KV head h >> row_shift.

// SCORE + TOPK with the group's per-head scores added instead of maximised (one cluster per unit, no scratch);
// per_head: no reduction at all, one list per QUERY head (idx, count, hist_out then have n_q_heads rows per sequence).
cudaError_t launch_score_topk_sum(int B, int Hq, int Hkv, const uint32_t *q_codes, const uint32_t *k_codes, long long kc_sb,
                                  long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq, int k_uniform,
                                  int k_max, int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                                  int32_t *hist_out, cudaStream_t st, Windows win = Windows{0, 0}, bool per_head = false);

cudaError_t launch_attention(bool gather, int B, int Hq, int Hkv, float sm_scale, const uint16_t *q,
                             TensorView K, TensorView V, const int32_t *seq_lens, const int32_t *idx,
                             long long idx_sb, long long idx_sh, const int32_t *count, int max_items,
                             uint16_t *out, float *lse, float *part_ml, float *part_acc, int32_t *tickets,
                             uint32_t *status, cudaStream_t st, int count_from_k = 0,
                             const int32_t *k_per_seq = nullptr, int k_uniform = 0, Windows win = Windows{0, 0},
                             const int32_t *block_table = nullptr, long long bt_sb = 0, int page_shift = 0,
                             int kv_shift = 0);   // kv_shift: unit head h reads K/V head h >> kv_shift

// The whole layer-step in one launch (one cluster per unit); only for small batches.  v_new_host != NULL: q,
// k_new and v_new are mapped host memory and the kernel appends the new K/V rows itself (host-buffer entry).
bool fused_step_eligible(int B, int Hq, int Hkv, int max_seq_len, int k_max);
bool fused_step_from_host_eligible(int B, int Hq, int Hkv, int max_seq_len, int k_max);   // ... with mapped host inputs
cudaError_t launch_fused_step(int B, int Hq, int Hkv, float sm_scale, const MapView &map_q, const MapView &map_k,
                              const uint16_t *q, const uint16_t *k_new, TensorView K, TensorView V, uint32_t *k_codes,
                              long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq,
                              int k_uniform, int max_seq_len, int k_max, uint32_t *q_codes, int32_t *idx,
                              long long idx_sb, long long idx_sh, int32_t *count, uint16_t *out, float *lse,
                              cudaStream_t st, Windows win = Windows{0, 0}, const int32_t *block_table = nullptr,
                              long long bt_sb = 0, int page_shift = 0, const uint16_t *v_new_host = nullptr);

// SCORE + TOPK and GATHER-ATT of a step in one persistent kernel whose SCORE warps run ahead of its GATHER warps
// (steps of more units than the single-cluster kernel holds; the query signatures come from ENCODE in front).
bool pipe_step_eligible(int B, int Hq, int Hkv);
cudaError_t launch_pipe_step(int B, int Hq, int Hkv, float sm_scale, const uint32_t *q_codes, const uint32_t *k_codes,
                             long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq, int k_uniform,
                             int max_seq_len, int k_max, int32_t *idx, long long idx_sb, long long idx_sh, int32_t *count,
                             const uint16_t *q, TensorView K, TensorView V, uint16_t *out, float *lse, int32_t *tickets,
                             int32_t *s1_done, int32_t *s2_done, int32_t *ws_hist, unsigned char *ws_scores, long long score_row,
                             float *part_ml, float *part_acc, uint32_t *status, cudaStream_t st, Windows win = Windows{0, 0},
                             const int32_t *block_table = nullptr, long long bt_sb = 0, int page_shift = 0);

// Stand-alone GATHER-ATT with one 8-CTA cluster per unit (few units, short lists).
bool gather_cluster_eligible(int B, int Hq, int Hkv, int k_max);
cudaError_t launch_gather_cluster(int B, int Hq, int Hkv, float sm_scale, const uint16_t *q, TensorView K, TensorView V,
                                  const int32_t *seq_lens, const int32_t *idx, long long idx_sb, long long idx_sh,
                                  const int32_t *count, int k_max, uint16_t *out, float *lse, uint32_t *status,
                                  cudaStream_t st, const int32_t *block_table = nullptr, long long bt_sb = 0,
                                  int page_shift = 0);

// Signatures of 64 .. 512 bits through ENCODE and SCORE + TOPK (packed 64-bit words; strides in words).
cudaError_t launch_encode_wide(const MapView &map, int n_bits, int heads_per_kv, TensorView x, int B, int H, int T,
                               uint64_t *codes, long long c_sb, long long c_sh, const int32_t *slot, cudaStream_t st);
size_t wide_workspace_bytes(int B, int Hkv, int max_seq_len);
cudaError_t launch_score_topk_wide(int B, int Hq, int Hkv, int n_bits, const uint64_t *q_codes, const uint64_t *k_codes,
                                   long long kc_sb, long long kc_sh, const int32_t *seq_lens, const int32_t *k_per_seq,
                                   int k_uniform, int max_seq_len, int k_max, int32_t *idx, long long idx_sb, long long idx_sh,
                                   int32_t *count, int32_t *hist_out, void *workspace, cudaStream_t st, Windows win);

cudaError_t launch_score_wide(const uint64_t *q_code, const uint64_t *k_codes, long long n, int n_words, uint16_t *scores,
                              cudaStream_t st);
cudaError_t launch_inner_products(const uint16_t *q, const uint16_t *K, long long n, long long row_stride, float *dots,
                                  cudaStream_t st);

cudaError_t launch_append_kv(int B, int Hq, int Hkv, const uint16_t *k_new, const uint16_t *v_new, TensorView K,
                             TensorView V, const int32_t *seq_lens, const uint16_t *q_src, uint16_t *q_dst,
                             uint16_t *k_dst, cudaStream_t st, const int32_t *block_table = nullptr, long long bt_sb = 0,
                             int page_shift = 0);

} // namespace ha
