/*
 * hashattn.h — C ABI of the B200 (sm_100a) HashAttention decode library.
 *
 * The library implements the decode-time sparse-attention recipe of the HashAttention paper
 * (arXiv 2412.14468, Section 4): ENCODE the query and the newly appended key into 32-bit
 * signatures with the learned mappings (Eq. 2), SCORE every cached token by the Hamming
 * distance between signatures (Eq. 1, computed as bitcount(xor), Section 4.1
 * "Implementation"), take the standard TOPK per KV head, and run GATHER-ATT — exact softmax
 * attention restricted to the selected tokens (Section 4), reading K/V rows by index without
 * compacting them (Section 4.4).
 *
 * General conventions
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller and
 *     must stay valid until the work enqueued on `stream` has completed.  bf16 values are passed
 *     as uint16_t bit patterns.  `stream` is a cudaStream_t passed as void* (NULL = legacy
 *     default stream).
 *   - Calls only enqueue work on `stream`: no host synchronisation and no allocation, except
 *     where stated (ha_read_device_status, ha_sparse_decode_host, ha_sparse_decode_paged_host).
 *   - Scratch memory is one caller-owned workspace of at least ha_workspace_bytes(...) bytes,
 *     256-byte aligned, prepared once with ha_workspace_init.  Calls that share a workspace must
 *     be ordered on one stream.
 *   - Kernels are launched with programmatic stream serialization: a kernel may start while its
 *     predecessor in the stream is finishing, and reads seq_lens, k_per_seq and the key signatures
 *     before it waits for that predecessor.  This is safe behind ordinary kernels and copies (they
 *     complete before anything of this library starts) and between calls of this library: the only
 *     signatures a library kernel directly in front may still be writing are those of the appended
 *     tokens, i.e. slot seq_len-1 (ha_encode with slot[b] = seq_len[b]-1, or this step's own k_new)
 *     and slot seq_len-2 (a layer-step on the same cache for a sequence one token shorter), and every
 *     scanning kernel reads these again after its wait.  A caller whose own preceding kernel both
 *     writes those arrays AND releases its dependents early (griddepcontrol.launch_dependents) must
 *     release them only after the writes.
 *   - seq_lens[b] <= max_seq_len (where a call takes max_seq_len) and seq_lens[b] <= the number of
 *     token slots of K, V and k_codes are the caller's promise.  SCORE + TOPK clamps a longer
 *     sequence to max_seq_len; the append of the host-buffer entries and GATHER-ATT do not clamp.
 *   - Return value: HA_OK, or an HA_ERR_* code for errors detectable on the host (nothing is
 *     enqueued in that case).  Errors only visible on the device (an index outside the sequence)
 *     set a bit in the workspace status word, are skipped, and never trap.
 *   - Fixed by the method's configuration (Section 5.2; abstract): head_dim = 128, signature
 *     width b = 32 bits, mapping network 128x128 - 128x128 - 128x32.  Other values return
 *     HA_ERR_UNSUPPORTED, except in the entry points named *_wide, which take b = 64 .. 512.  n_q_heads must be a multiple of n_kv_heads with a group size
 *     G = n_q_heads / n_kv_heads <= 8; query head j uses KV head j / G.
 */
#ifndef HASHATTN_H
#define HASHATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HA_OK 0
#define HA_ERR_INVALID_ARG 1 /* NULL where a pointer is required, negative size, bad stride */
#define HA_ERR_UNSUPPORTED 2 /* head_dim != 128, n_bits != 32, group size > 8, ... */
#define HA_ERR_WORKSPACE 3   /* workspace NULL, misaligned or smaller than ha_workspace_bytes */
#define HA_ERR_CUDA 4        /* a CUDA runtime call failed (launch error, bad stream) */
#define HA_ERR_STATIC_LIMIT 5 /* ha_gather_attn_static: problem larger than the library's built-in scratch */

/* bits of the device status word (ha_read_device_status) */
#define HA_DEV_BAD_INDEX 1u /* an idx entry >= seq_len was met and skipped */
#define HA_DEV_TIMEOUT 2u   /* a bounded wait inside a kernel gave up (ha_encode_prefill's tensor-core path,
                               ha_sparse_decode_pipelined); the kernel returned early and its outputs are not valid */

#define HA_HEAD_DIM 128
#define HA_N_BITS 32
#define HA_HIST_BINS 33 /* scores 0..32 */

/* Problem shape of one layer-step. sm_scale multiplies the logits (1/sqrt(d) in the SDPA
 * definition, Section 3.1).
 * n_sink / n_local: the first n_sink and the most recent n_local tokens of every sequence are always
 * in context, and the budget k counts the heavy tokens retrieved in addition among the others
 * (Section 5, paragraph on baselines, where both are 128).  0 / 0 is the plain top-k of Section 4.
 * Only SCORE + TOPK (ha_score_topk, ha_sparse_decode, ha_sparse_decode_host) looks at them. */
typedef struct ha_shape {
    int32_t batch;
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t head_dim; /* must be 128 */
    float sm_scale;
    int32_t n_sink;   /* >= 0 */
    int32_t n_local;  /* >= 0 */
} ha_shape;

/* One side's mapping networks (phi_q or phi_kv of Eq. 2), one network per KV head.
 * y = x W + b with W stored [in][out] row-major; hidden activation ReLU; bit o of the signature
 * is 1 iff output o of the last layer is > 0.  Biases may be NULL (= zeros). */
typedef struct ha_mapping {
    int32_t n_kv_heads;
    int32_t in_dim;  /* 128 */
    int32_t hid_dim; /* 128 */
    int32_t n_bits;  /* 32 */
    const uint16_t *w1; /* bf16 [n_kv_heads][128][128] */
    const uint16_t *w2; /* bf16 [n_kv_heads][128][128] */
    const uint16_t *w3; /* bf16 [n_kv_heads][128][32]  */
    const float *b1;    /* fp32 [n_kv_heads][128] or NULL */
    const float *b2;    /* fp32 [n_kv_heads][128] or NULL */
    const float *b3;    /* fp32 [n_kv_heads][32]  or NULL */
} ha_mapping;

/* A bf16 tensor [batch][heads][tokens][128] addressed by element strides; the last dimension is
 * contiguous and every row must start on a 16-byte boundary (strides multiples of 8). */
typedef struct ha_tensor {
    const void *ptr;
    int64_t stride_b;
    int64_t stride_h;
    int64_t stride_n;
} ha_tensor;

/* Bytes of workspace needed by every entry point for shapes up to (shape, max_seq_len, max_k).
 * Returns 0 if the shape is unsupported.  The size depends on the batch, the head counts and
 * max_seq_len; max_k (>= 0) is checked but does not enter the size, because index lists are the
 * caller's own buffers. */
size_t ha_workspace_bytes(const ha_shape *shape, int32_t max_seq_len, int32_t max_k);

/* Clears the workspace header (device status word).  Call once after allocating the workspace
 * and whenever the status should be reset. */
int ha_workspace_init(void *workspace, size_t ws_bytes, void *stream);

/* ENCODE — Eq. 2: codes = pack(sign(F(x)) > 0) with F the Section 5.2 network; phi_kv takes the
 * key only (Section 4.1).  Arithmetic: fp32 fused multiply-add chain per output, ascending input
 * index, started from the bias; hidden activations stay fp32.
 *   x             bf16 [batch][n_heads][n_tokens][128] (strides in x)
 *   heads_per_kv  head h uses network h / heads_per_kv (G for the query side, 1 for the key side)
 *   codes         out: codes[b*c_stride_b + h*c_stride_h + t] for t < n_tokens, or, when `slot`
 *                 is given (n_tokens must be 1), codes[b*c_stride_b + h*c_stride_h + slot[b]]
 *                 (the append of Section 4.1: slot[b] = seq_len[b] - 1); slot[b] < 0 skips b. */
int ha_encode(const ha_mapping *map, int32_t heads_per_kv, const ha_tensor *x, int32_t batch,
              int32_t n_heads, int32_t n_tokens, uint32_t *codes, int64_t c_stride_b,
              int64_t c_stride_h, const int32_t *slot, void *stream);

/* ENCODE of whole prompts on the tensor cores — the signature cache of n_tokens tokens per head at
 * once (Section 4.1 "Implementation": signatures are computed and cached along with the KV cache;
 * Section 5.2 names these matrix multiplications as the latency bottleneck at short contexts).
 * Arguments as ha_encode without `slot`.  The three layers run as bf16 tensor-core GEMMs with fp32
 * accumulation; hidden activations enter the next layer as a bf16 pair hi + lo.  The sums are
 * therefore NOT the fused-multiply-add chain of ha_encode: a signature bit may differ from
 * ha_encode's where the exact last-layer output lies within about 1e-5 of zero, and is identical
 * everywhere else.  Use ha_encode where bit-exact agreement with the decode step matters.
 *   path       HA_PREFILL_TCGEN05: tcgen05.mma with the accumulators and the hidden activations in
 *              tensor memory; HA_PREFILL_MMA_SYNC: warp-level mma.sync with the activations chained
 *              through registers (the earlier tensor-core generation's path, kept for comparison)
 *   workspace  optional (may be NULL): a workspace from ha_workspace_bytes; if the tcgen05 kernel
 *              gives up waiting for its tensor cores it raises HA_DEV_TIMEOUT in its status word */
#define HA_PREFILL_TCGEN05 0
#define HA_PREFILL_MMA_SYNC 1
int ha_encode_prefill(const ha_mapping *map, int32_t heads_per_kv, const ha_tensor *x, int32_t batch,
                      int32_t n_heads, int32_t n_tokens, uint32_t *codes, int64_t c_stride_b,
                      int64_t c_stride_h, int32_t path, void *workspace, void *stream);

/* SCORE + TOPK — Eq. 1 as s = 32 - bitcount(k_code xor q_code) (Section 4.1), group score =
 * max over the G query heads of the KV head, then the standard top-k (Section 4) with ties
 * broken towards the lowest token index.
 *   q_codes    u32 [batch][n_q_heads]
 *   k_codes    u32 [batch][n_kv_heads][>= seq_len], token-contiguous, rows 16-byte aligned
 *   seq_lens   i32 [batch]
 *   k_per_seq  i32 [batch] or NULL (then k_uniform is used for every sequence)
 *   idx        out i32 [batch][n_kv_heads][k_max] (strides given), ascending token index,
 *              entries count..k_max-1 set to -1; k_max = max budget = the k passed to
 *              ha_workspace_bytes or less
 *   count      out i32 [batch][n_kv_heads] = min(k_b, seq_len_b)
 *   hist_out   optional out i32 [batch][n_kv_heads][33]: histogram of the group scores
 * With shape->n_sink or shape->n_local > 0: tokens [0, n_sink) and [seq_len - n_local, seq_len) are
 * always selected, k_b more come from the others by the same order; count = windows + min(k_b, others);
 * hist_out covers the others only; k_max must be >= n_sink + n_local (else HA_ERR_INVALID_ARG) and
 * should be >= n_sink + n_local + max k_b, since the budget is cut to what fits in k_max. */
int ha_score_topk(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes,
                  int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens,
                  const int32_t *k_per_seq, int32_t k_uniform, int32_t max_seq_len, int32_t k_max,
                  int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                  int32_t *hist_out, void *workspace, size_t ws_bytes, void *stream);

/* SCORE + TOPK with the other reduction over a GQA group: the per-head scores of Eq. 1 (as 32 - bitcount(k_code
 * xor q_code), Section 4.1) ADDED over the G query heads of the KV head, range 0 .. 32 G, then the standard top-k
 * of Section 4 with ties towards the lowest token index.  The paper defines the score for one query head; the
 * layer-step (ha_sparse_decode, ha_score_topk) takes the maximum over the group, this entry is the stand-alone
 * alternative and equals ha_score_topk when G = 1.  Arguments, layouts, windows (shape->n_sink / n_local) and
 * the idx / count outputs as in ha_score_topk; no workspace and no maximum sequence length are needed (any
 * seq_len >= 0), and
 *   hist_out   optional out i32 [batch][n_kv_heads][32 G + 1]: histogram of the summed scores (windows excluded).
 * The index lists feed ha_gather_attn unchanged.  A plain launch on `stream`; it can be captured into a CUDA graph after
 * one call outside capture (which sets the kernel's attributes on this device). */
int ha_score_topk_sum(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes,
                      int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens,
                      const int32_t *k_per_seq, int32_t k_uniform, int32_t k_max, int32_t *idx,
                      int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, int32_t *hist_out,
                      void *stream);

/* SCORE + TOPK and GATHER-ATT with one index list per QUERY head: no reduction over a GQA group at all.  Query head j
 * scores the signatures of its KV head j / G by Eq. 1 (Section 4.1) and keeps its own top-k (Section 4), exactly what
 * the paper defines for one head; GATHER-ATT then reads the K/V rows of KV head j / G through query head j's list, so
 * the K/V traffic is G times that of the grouped entries.
 *   ha_score_topk_per_head   arguments as ha_score_topk_sum, except
 *       idx        out i32 [batch][n_q_heads][k_max] (strides given; idx_stride_h steps over QUERY heads)
 *       count      out i32 [batch][n_q_heads]
 *       hist_out   optional out i32 [batch][n_q_heads][33]
 *     batch * n_q_heads must not exceed 65536 (else HA_ERR_UNSUPPORTED).
 *   ha_gather_attn_per_head  arguments as ha_gather_attn with idx / count as above (contiguous K/V only); the
 *     workspace must come from ha_workspace_bytes for the shape with n_kv_heads set to n_q_heads. */
int ha_score_topk_per_head(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes,
                           int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens,
                           const int32_t *k_per_seq, int32_t k_uniform, int32_t k_max, int32_t *idx,
                           int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, int32_t *hist_out,
                           void *stream);
int ha_gather_attn_per_head(const ha_shape *shape, const uint16_t *q, const ha_tensor *K,
                            const ha_tensor *V, const int32_t *seq_lens, const int32_t *idx,
                            int64_t idx_stride_b, int64_t idx_stride_h, const int32_t *count,
                            int32_t k_max, uint16_t *out, float *lse, void *workspace, size_t ws_bytes,
                            void *stream);

/* GATHER-ATT — Section 4: out_j = sum_{i in I} softmax_I(sm_scale <q_j, k_i>) v_i for every
 * query head j, I = idx[b][j / G][0..count).  K/V rows are read in place through the indices
 * (Section 4.4).  fp32 accumulation, one rounding to bf16.
 *   idx entries < 0 are padding and skipped; entries >= seq_len are skipped and raise
 *   HA_DEV_BAD_INDEX.  An empty list gives out = 0, lse = -inf.
 *   out bf16 [batch][n_q_heads][128]; lse fp32 [batch][n_q_heads] or NULL. */
int ha_gather_attn(const ha_shape *shape, const uint16_t *q, const ha_tensor *K,
                   const ha_tensor *V, const int32_t *seq_lens, const int32_t *idx,
                   int64_t idx_stride_b, int64_t idx_stride_h, const int32_t *count, int32_t k_max,
                   uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream);

/* GATHER-ATT over a paged K/V cache (Section 4.4: K/V rows are read in place through the indices; the
 * paper's vLLM integration keeps K/V in pages addressed through a block table).  Same computation and
 * arguments as ha_gather_attn, except that token t of sequence b is found in page
 * block_table[b * bt_stride_b + t / page_size] at slot t % page_size:
 *   K_pool, V_pool  bf16 rows [n_pages][n_kv_heads][page_size][128] described by (stride_b = page stride,
 *                   stride_h = head stride, stride_n = slot stride), elements; both pools must have the same
 *                   number of rows per page stride (stride_b / stride_n, an integer)
 *   block_table     i32 [batch][>= ceil(seq_len / page_size)] page numbers (device)
 *   page_size       power of two (1 = every token its own page)
 * The index lists hold logical token numbers, exactly as ha_score_topk writes them (here the signature cache
 * stays one contiguous array per sequence and KV head; the *_paged entries further down page it too). */
int ha_gather_attn_paged(const ha_shape *shape, const uint16_t *q, const ha_tensor *K_pool,
                         const ha_tensor *V_pool, const int32_t *block_table, int64_t bt_stride_b,
                         int32_t page_size, const int32_t *seq_lens, const int32_t *idx,
                         int64_t idx_stride_b, int64_t idx_stride_h, const int32_t *count, int32_t k_max,
                         uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream);

/* Dense decode attention — single-query SDPA over all seq_len tokens (Section 3.1): the
 * computation the sparse path replaces, provided as the same-run comparator. */
int ha_dense_decode(const ha_shape *shape, const uint16_t *q, const ha_tensor *K,
                    const ha_tensor *V, const int32_t *seq_lens, int32_t max_seq_len,
                    uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream);

/* One whole layer-step (Section 4 recipe; Section 4.1 "Implementation"): signature of the new
 * key appended at slot seq_len-1 (skipped if k_new is NULL), query signatures, SCORE, TOPK,
 * GATHER-ATT.  Same semantics as ha_encode (x2) + ha_score_topk + ha_gather_attn.
 *   k_new    bf16 [batch][n_kv_heads][128] contiguous or NULL
 *   q_codes  out u32 [batch][n_q_heads]; k_codes is read and, if k_new, written at the slot. */
int ha_sparse_decode(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                     const uint16_t *q, const uint16_t *k_new, const ha_tensor *K,
                     const ha_tensor *V, uint32_t *k_codes, int64_t kc_stride_b,
                     int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                     int32_t k_uniform, int32_t max_seq_len, int32_t k_max, uint32_t *q_codes,
                     int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                     uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream);

/* The same layer-step (Section 4 recipe; Section 4.1 "Implementation") on another schedule: ENCODE, then ONE persistent
 * kernel in which every SM's SCORE + TOPK warps run ahead of its GATHER-ATT warps over a range of (sequence, KV head)
 * units, so that the bit counting of later units (Eq. 1) overlaps the K/V row fetch of earlier ones; units are released
 * to the GATHER-ATT warps through counters in the workspace.  Arguments, outputs and results as ha_sparse_decode
 * (signatures, counts and index lists bit-identical; outputs to fp32 reordering); contiguous K/V only;
 * batch * n_kv_heads <= 1024 (else HA_ERR_UNSUPPORTED).  If a wait inside the kernel runs out (it never should: all
 * CTAs are resident at once) the kernel ends early, raises HA_DEV_TIMEOUT in the workspace status word and the outputs
 * must not be used; call ha_workspace_init before the workspace is used again.
 * On B200 ha_sparse_decode is the faster of the two at every shape measured so far: scoring needs most of an SM's warp
 * slots to keep its population-count unit busy, which the row fetch's registers and shared memory do not leave. */
int ha_sparse_decode_pipelined(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                               const uint16_t *q, const uint16_t *k_new, const ha_tensor *K, const ha_tensor *V,
                               uint32_t *k_codes, int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens,
                               const int32_t *k_per_seq, int32_t k_uniform, int32_t max_seq_len, int32_t k_max,
                               uint32_t *q_codes, int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h,
                               int32_t *count, uint16_t *out, float *lse, void *workspace, size_t ws_bytes,
                               void *stream);

/* One whole layer-step over a paged K/V cache: ha_sparse_decode with K/V addressed as in
 * ha_gather_attn_paged (pools + block table + page_size); the signature cache k_codes stays contiguous. */
int ha_sparse_decode_paged(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                           const uint16_t *q, const uint16_t *k_new, const ha_tensor *K_pool,
                           const ha_tensor *V_pool, const int32_t *block_table, int64_t bt_stride_b,
                           int32_t page_size, uint32_t *k_codes, int64_t kc_stride_b, int64_t kc_stride_h,
                           const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                           int32_t max_seq_len, int32_t k_max, uint32_t *q_codes, int32_t *idx,
                           int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, uint16_t *out,
                           float *lse, void *workspace, size_t ws_bytes, void *stream);

/* The same layer-step driven from HOST buffers (the per-step inputs of a decoder: the new
 * query, key and value vectors; Section 4.1): copies q_host, k_new_host, v_new_host to the device
 * (staging inside the workspace), writes the new K/V rows into the resident cache at slot
 * seq_len-1, runs ha_sparse_decode, copies `out` back to out_host and SYNCHRONISES the stream.
 * Host buffers should be pinned: buffers that the device can address (cudaHostAlloc / cudaHostRegister
 * under unified addressing) are read and written by the kernels themselves, without staged copies, and
 * when the step is one fused launch with lists of up to 2048 entries that kernel also appends the new
 * rows; any other buffer goes through staged cudaMemcpyAsync calls.  The result is the same in every case.
 * K, V, k_codes, seq_lens, k_per_seq, idx, count stay device pointers (resident state).  K and V must
 * be writable. */
int ha_sparse_decode_host(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                          const uint16_t *q_host, const uint16_t *k_new_host,
                          const uint16_t *v_new_host, const ha_tensor *K, const ha_tensor *V,
                          uint32_t *k_codes, int64_t kc_stride_b, int64_t kc_stride_h,
                          const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                          int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                          int64_t idx_stride_h, int32_t *count, uint16_t *out_host,
                          void *workspace, size_t ws_bytes, void *stream);

/* ha_sparse_decode_host over a paged K/V cache (pools + block table + page_size as in ha_gather_attn_paged): the
 * new K/V rows of sequence b go to slot (seq_len - 1) % page_size of page block_table[b][(seq_len - 1) / page_size],
 * which the caller must have allocated; everything else as ha_sparse_decode_host. */
int ha_sparse_decode_paged_host(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                                const uint16_t *q_host, const uint16_t *k_new_host,
                                const uint16_t *v_new_host, const ha_tensor *K_pool,
                                const ha_tensor *V_pool, const int32_t *block_table, int64_t bt_stride_b,
                                int32_t page_size, uint32_t *k_codes, int64_t kc_stride_b,
                                int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                                int32_t k_uniform, int32_t max_seq_len, int32_t k_max, int32_t *idx,
                                int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                                uint16_t *out_host, void *workspace, size_t ws_bytes, void *stream);

/* The signature cache in pages as well (Section 4.1 "Implementation": signatures are computed and cached along with the
 * KV cache; the paper's vLLM integration, Section 4.4, keeps that cache in pages).  code_pool holds the 32-bit signatures
 * as [n_pages][n_kv_heads][page_size] addressed by element strides (cp_stride_page, cp_stride_head; multiples of 4 and a
 * 16-byte aligned base when page_size >= 4), with the SAME block table and page size as the K/V pools: the signature of
 * token t of sequence b and KV head h is
 *     code_pool[block_table[b * bt_stride_b + t / page_size] * cp_stride_page + h * cp_stride_head + t % page_size].
 * page_size is a power of two; 16 makes a page one 64-byte segment per head, 1 gives every token its own page.
 * Index lists hold logical token numbers and are bit-identical to those over a contiguous cache.
 *   ha_score_topk_paged            ha_score_topk over the pool (arguments otherwise the same)
 *   ha_score_topk_per_head_paged   ha_score_topk_per_head over the pool; unlike its contiguous form it takes
 *                                  max_seq_len and a workspace from ha_workspace_bytes for the shape with n_kv_heads
 *                                  set to n_q_heads
 *   ha_gather_attn_per_head_paged  ha_gather_attn_per_head over paged K/V pools (as ha_gather_attn_paged)
 *   ha_encode_append_paged         the append of Section 4.1 into the pool: signature of k_new [batch][n_kv_heads][128]
 *                                  (phi_kv) written at token seq_lens[b] - 1 of sequence b (skipped if that is < 0)
 *   ha_sparse_decode_paged_codes   the whole layer-step with K, V and the signatures all paged (ENCODE with the append
 *                                  into the pool, SCORE + TOPK, GATHER-ATT as separate kernels) */
int ha_score_topk_paged(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *code_pool, int64_t cp_stride_page,
                        int64_t cp_stride_head, const int32_t *block_table, int64_t bt_stride_b, int32_t page_size,
                        const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform, int32_t max_seq_len,
                        int32_t k_max, int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                        int32_t *hist_out, void *workspace, size_t ws_bytes, void *stream);
int ha_score_topk_per_head_paged(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *code_pool,
                                 int64_t cp_stride_page, int64_t cp_stride_head, const int32_t *block_table,
                                 int64_t bt_stride_b, int32_t page_size, const int32_t *seq_lens, const int32_t *k_per_seq,
                                 int32_t k_uniform, int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                                 int64_t idx_stride_h, int32_t *count, int32_t *hist_out, void *workspace, size_t ws_bytes,
                                 void *stream);
int ha_gather_attn_per_head_paged(const ha_shape *shape, const uint16_t *q, const ha_tensor *K_pool,
                                  const ha_tensor *V_pool, const int32_t *block_table, int64_t bt_stride_b,
                                  int32_t page_size, const int32_t *seq_lens, const int32_t *idx, int64_t idx_stride_b,
                                  int64_t idx_stride_h, const int32_t *count, int32_t k_max, uint16_t *out, float *lse,
                                  void *workspace, size_t ws_bytes, void *stream);
int ha_encode_append_paged(const ha_mapping *map, const uint16_t *k_new, int32_t batch, uint32_t *code_pool,
                           int64_t cp_stride_page, int64_t cp_stride_head, const int32_t *block_table, int64_t bt_stride_b,
                           int32_t page_size, const int32_t *seq_lens, void *stream);
int ha_sparse_decode_paged_codes(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k, const uint16_t *q,
                                 const uint16_t *k_new, const ha_tensor *K_pool, const ha_tensor *V_pool,
                                 uint32_t *code_pool, int64_t cp_stride_page, int64_t cp_stride_head,
                                 const int32_t *block_table, int64_t bt_stride_b, int32_t page_size, const int32_t *seq_lens,
                                 const int32_t *k_per_seq, int32_t k_uniform, int32_t max_seq_len, int32_t k_max,
                                 uint32_t *q_codes, int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                                 uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream);

/* GATHER-ATT without a caller-provided workspace.  (The paper has no counterpart of this entry
 * point; it exists for integration reasons only.)
 *
 * Some callers cannot give this library scratch memory because they cannot allocate device memory
 * at the point where they call it: a serving process that handed the whole GPU to its own memory
 * pool at start-up and has no hook to carve a buffer out of it for a third-party library, a
 * plug-in that is invoked from inside another runtime's operator callback where only kernel
 * launches are permitted, or a latency-critical loop that must not risk the implicit device
 * synchronisation of cudaMalloc/cudaFree.  For them this variant of ha_gather_attn keeps the
 * split-K states, the ticket counters and the status word in a fixed array inside the library's
 * device image (about 2.4 MB, held by every GPU that loads the library until the process exits).
 * It calls no cudaMalloc, cudaFree or other allocating routine; inputs and outputs are still the
 * caller's.  Same arguments and results as ha_gather_attn, minus the workspace.
 *
 * Limits: batch * n_kv_heads <= 64, and a GPU with at most 256 SMs; anything larger returns
 * HA_ERR_STATIC_LIMIT and enqueues nothing.
 * First call on a device: looks up the array's device address (once per device, that device must
 * be current); make that first call before any stream capture begins.
 * Sharing: every call on a device uses the same array and finds in it what the previous call left;
 * the call clears the words that must start at zero itself.  Two calls that can overlap on the
 * GPU (different streams without ordering) race on the array: order them.
 * An index outside its sequence is skipped as in ha_gather_attn; the status word it would flag is
 * internal to the array and not readable through this entry point. */
int ha_gather_attn_static(const ha_shape *shape, const uint16_t *q, const ha_tensor *K,
                          const ha_tensor *V, const int32_t *seq_lens, const int32_t *idx,
                          int64_t idx_stride_b, int64_t idx_stride_h, const int32_t *count,
                          int32_t k_max, uint16_t *out, float *lse, void *stream);

/* SCORE for wide signatures (Section "Latency of SCORE computation" and its table: Hamming distance on
 * packed 64-bit integers, 64 to 512 bits per token; Eq. 1 with the bitcount identity of Section 4.1 at
 * b bits).  scores[i] = n_bits - popcount(k_codes[i] xor q_code), 0 <= i < n.
 *   q_code   device, n_bits / 64 words; bit j of a signature is bit j % 64 of word j / 64.
 *   k_codes  device, [n][n_bits / 64] words, contiguous, 16-byte aligned.
 *   scores   device, n 16-bit values, 4-byte aligned; written by the call, owned by the caller.
 * n_bits must be 64, 128, 256 or 512 (HA_ERR_UNSUPPORTED otherwise); n = 0 returns HA_OK without a
 * launch; null or misaligned pointers and n < 0 give HA_ERR_INVALID_ARG.  One query, no group
 * reduction, no selection: this is the stand-alone scoring pass that the paper times against the
 * inner product, not a step of ha_sparse_decode (whose signatures have 32 bits). */
int ha_score_wide(const uint64_t *q_code, const uint64_t *k_codes, int64_t n, int32_t n_bits,
                  uint16_t *scores, void *stream);

/* ENCODE -> SCORE -> TOPK at signatures of b = 64, 128, 256 or 512 bits (the widths of the paper's study of the number
 * of bits and of its SCORE-latency table, which keeps them as packed 64-bit integers).  The index lists and counts have
 * the layout of ha_score_topk's and feed ha_gather_attn unchanged.
 *
 * ha_encode_wide — Eq. 2 with a last layer of 128 x b: map->n_bits = b, map->w3 bf16 [n_kv_heads][128][b], map->b3 fp32
 *   [n_kv_heads][b] or NULL; layers 1 and 2, the arithmetic of every output (fp32 fused multiply-add chain, ascending
 *   input index, from the bias) and the arguments as ha_encode, except
 *   codes   out, 64-bit words [batch][n_heads][tokens][b / 64] (8-byte aligned; c_stride_b, c_stride_h in words); bit j
 *           of a signature is bit j % 64 of word j / 64; with `slot` (n_tokens == 1) the signature of sequence b goes
 *           to token slot[b] (slot[b] < 0 skips b).
 * ha_score_topk_wide — Eq. 1 as s = b - bitcount(k_code xor q_code) (Section 4.1), 0 .. b, group score = max over the
 *   G query heads of the KV head, then the standard top-k (Section 4), ties to the lowest token index; always-kept
 *   windows (shape->n_sink / n_local) as in ha_score_topk.
 *   q_codes   words [batch][n_q_heads][b / 64]
 *   k_codes   words [batch][n_kv_heads][>= seq_len][b / 64], 16-byte aligned (kc_stride_b, kc_stride_h in words)
 *   hist_out  optional out i32 [batch][n_kv_heads][b + 1]: histogram of the group scores (windows excluded)
 *   workspace at least ha_workspace_bytes_wide(shape, max_seq_len) bytes, 256-byte aligned; needs no initialisation;
 *             calls that share it must be ordered on one stream. */
int ha_encode_wide(const ha_mapping *map, int32_t heads_per_kv, const ha_tensor *x, int32_t batch, int32_t n_heads,
                   int32_t n_tokens, uint64_t *codes, int64_t c_stride_b, int64_t c_stride_h, const int32_t *slot,
                   void *stream);
size_t ha_workspace_bytes_wide(const ha_shape *shape, int32_t max_seq_len);
int ha_score_topk_wide(const ha_shape *shape, int32_t n_bits, const uint64_t *q_codes, const uint64_t *k_codes,
                       int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                       int32_t k_uniform, int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                       int64_t idx_stride_h, int32_t *count, int32_t *hist_out, void *workspace, size_t ws_bytes,
                       void *stream);

/* The comparator column of the same table: dots[i] = <q, K[i]> for one query and n keys of 128 bf16
 * components ("128 x 16Float"), fp32 accumulation.
 *   q     device, 128 bf16 values, 16-byte aligned.
 *   K     device, row i at K + i * row_stride (elements); row_stride >= 128 and a multiple of 8,
 *         base 16-byte aligned.
 *   dots  device, n fp32 values.
 * Errors as for ha_score_wide. */
int ha_inner_products(const uint16_t *q, const uint16_t *K, int64_t n, int64_t row_stride, float *dots,
                      void *stream);

/* Copies the device status word to *flags (host) and clears nothing; synchronises `stream`. */
int ha_read_device_status(void *workspace, void *stream, uint32_t *flags);

/* Number of kernels this library has launched in this process (host-side counter). */
uint64_t ha_kernel_launches(void);

const char *ha_status_string(int status);
const char *ha_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HASHATTN_H */
