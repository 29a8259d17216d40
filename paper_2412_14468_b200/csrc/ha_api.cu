// C-ABI entry points: argument validation, workspace carving, kernel sequencing.
// See include/hashattn.h for the contract of every function.
#include <atomic>

#include "ha_common.cuh"

namespace ha {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static int check_shape(const ha_shape *s) {
    if (!s) return HA_ERR_INVALID_ARG;
    if (s->batch < 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0) return HA_ERR_INVALID_ARG;
    if (s->head_dim != kD) return HA_ERR_UNSUPPORTED;
    if (s->n_q_heads % s->n_kv_heads != 0) return HA_ERR_UNSUPPORTED;
    const int G = s->n_q_heads / s->n_kv_heads;
    if (G != 1 && G != 2 && G != 4 && G != 8) return HA_ERR_UNSUPPORTED;
    if (s->n_kv_heads > 65535 || s->batch > 65535) return HA_ERR_UNSUPPORTED;
    if ((long long)s->n_kv_heads * s->batch > kMaxUnits) return HA_ERR_UNSUPPORTED;
    if (!(s->sm_scale == s->sm_scale)) return HA_ERR_INVALID_ARG;
    if (s->n_sink < 0 || s->n_local < 0) return HA_ERR_INVALID_ARG;
    return HA_OK;
}

static int check_mapping(const ha_mapping *m, int n_kv_heads) {
    if (!m || !m->w1 || !m->w2 || !m->w3) return HA_ERR_INVALID_ARG;
    if (m->in_dim != kD || m->hid_dim != kHid || m->n_bits != kBits) return HA_ERR_UNSUPPORTED;
    if (m->n_kv_heads <= 0 || (n_kv_heads > 0 && m->n_kv_heads != n_kv_heads)) return HA_ERR_INVALID_ARG;
    if (((uintptr_t)m->w1 | (uintptr_t)m->w2 | (uintptr_t)m->w3) & 15) return HA_ERR_INVALID_ARG;
    return HA_OK;
}

static int check_tensor(const ha_tensor *t) {
    if (!t || !t->ptr) return HA_ERR_INVALID_ARG;
    if (((uintptr_t)t->ptr & 15) || (t->stride_b & 7) || (t->stride_h & 7) || (t->stride_n & 7))
        return HA_ERR_INVALID_ARG;
    if (t->stride_n < kD) return HA_ERR_INVALID_ARG;
    return HA_OK;
}

// max_seq_len < 0: the call does not scan signatures and needs no score bytes
static int check_workspace(const ha_shape *s, int max_seq_len, void *ws, size_t bytes, WorkspaceLayout *L) {
    if (!ws || ((uintptr_t)ws & 255)) return HA_ERR_WORKSPACE;
    *L = make_layout(s->batch, s->n_q_heads, s->n_kv_heads, max_seq_len < 0 ? 0 : max_seq_len);
    if (bytes < L->total) return HA_ERR_WORKSPACE;
    return HA_OK;
}

static TensorView view(const ha_tensor *t) {
    return TensorView{reinterpret_cast<const uint16_t *>(t->ptr), (long long)t->stride_b, (long long)t->stride_h,
                      (long long)t->stride_n};
}

static MapView view(const ha_mapping *m) { return MapView{m->w1, m->w2, m->w3, m->b1, m->b2, m->b3}; }

template <typename T>
static T *ws_ptr(void *ws, size_t off) { return reinterpret_cast<T *>(reinterpret_cast<char *>(ws) + off); }

} // namespace ha

using namespace ha;

#define HA_TRY(expr)                      \
    do {                                  \
        int _st = (expr);                 \
        if (_st != HA_OK) return _st;     \
    } while (0)
#define HA_CUDA(expr)                              \
    do {                                           \
        if ((expr) != cudaSuccess) return HA_ERR_CUDA; \
    } while (0)

extern "C" {

size_t ha_workspace_bytes(const ha_shape *shape, int32_t max_seq_len, int32_t max_k) {
    if (check_shape(shape) != HA_OK || max_seq_len < 0 || max_k < 0) return 0;
    return make_layout(shape->batch, shape->n_q_heads, shape->n_kv_heads, max_seq_len).total;
}

int ha_workspace_init(void *workspace, size_t ws_bytes, void *stream) {
    if (!workspace || ((uintptr_t)workspace & 255) || ws_bytes < kHeaderBytes) return HA_ERR_WORKSPACE;
    // status and abort words, the ticket counters and the release counters (which every call leaves at zero again)
    size_t n = kHeaderBytes + (size_t)3 * kMaxUnits * 4;
    if (n > ws_bytes) n = ws_bytes;
    HA_CUDA(cudaMemsetAsync(workspace, 0, n, (cudaStream_t)stream));
    return HA_OK;
}

int ha_encode(const ha_mapping *map, int32_t heads_per_kv, const ha_tensor *x, int32_t batch, int32_t n_heads,
              int32_t n_tokens, uint32_t *codes, int64_t c_stride_b, int64_t c_stride_h, const int32_t *slot,
              void *stream) {
    HA_TRY(check_mapping(map, 0));
    HA_TRY(check_tensor(x));
    if (!codes || batch < 0 || n_heads <= 0 || n_tokens < 0 || heads_per_kv <= 0) return HA_ERR_INVALID_ARG;
    if (n_heads % heads_per_kv != 0 || n_heads / heads_per_kv != map->n_kv_heads) return HA_ERR_INVALID_ARG;
    if (slot && n_tokens != 1) return HA_ERR_INVALID_ARG;
    if (slot && heads_per_kv > 8) return HA_ERR_UNSUPPORTED;
    if (batch > 65535 || n_heads > 65535) return HA_ERR_UNSUPPORTED;
    if (batch == 0 || n_tokens == 0) return HA_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (n_tokens == 1 && heads_per_kv <= 8) {
        EncodeJob a{};
        a.x = reinterpret_cast<const uint16_t *>(x->ptr);
        a.x_sb = x->stride_b; a.x_sh = x->stride_h;
        a.codes = codes; a.c_sb = c_stride_b; a.c_sh = c_stride_h;
        a.slot = slot; a.slot_minus_one = 0;
        a.n_heads = n_heads; a.heads_per_kv = heads_per_kv; a.n_cta = batch * (n_heads / heads_per_kv);
        a.map = view(map);
        EncodeJob none{};
        HA_CUDA(launch_encode_vectors(a, none, st));
    } else {
        HA_CUDA(launch_encode_bulk(view(map), heads_per_kv, view(x), batch, n_heads, n_tokens, codes, c_stride_b,
                                   c_stride_h, st));
    }
    return HA_OK;
}

int ha_encode_prefill(const ha_mapping *map, int32_t heads_per_kv, const ha_tensor *x, int32_t batch, int32_t n_heads,
                      int32_t n_tokens, uint32_t *codes, int64_t c_stride_b, int64_t c_stride_h, int32_t path,
                      void *workspace, void *stream) {
    HA_TRY(check_mapping(map, 0));
    HA_TRY(check_tensor(x));
    if (!codes || batch < 0 || n_heads <= 0 || n_tokens < 0 || heads_per_kv <= 0) return HA_ERR_INVALID_ARG;
    if (n_heads % heads_per_kv != 0 || n_heads / heads_per_kv != map->n_kv_heads) return HA_ERR_INVALID_ARG;
    if (path != HA_PREFILL_TCGEN05 && path != HA_PREFILL_MMA_SYNC) return HA_ERR_INVALID_ARG;
    if (workspace && ((uintptr_t)workspace & 255)) return HA_ERR_WORKSPACE;
    if (batch == 0 || n_tokens == 0) return HA_OK;
    if (path == HA_PREFILL_MMA_SYNC)
        HA_CUDA(launch_encode_tc(view(map), heads_per_kv, view(x), batch, n_heads, n_tokens, codes, c_stride_b, c_stride_h,
                                 (cudaStream_t)stream));
    else
        HA_CUDA(launch_encode_umma(view(map), heads_per_kv, view(x), batch, n_heads, n_tokens, codes, c_stride_b,
                                   c_stride_h, reinterpret_cast<uint32_t *>(workspace), (cudaStream_t)stream));
    return HA_OK;
}

static int check_score_args(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes,
                            int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens, int32_t k_uniform,
                            const int32_t *k_per_seq, int32_t max_seq_len, int32_t k_max, int32_t *idx,
                            int32_t *count) {
    HA_TRY(check_shape(shape));
    if (!q_codes || !k_codes || !seq_lens || !idx || !count) return HA_ERR_INVALID_ARG;
    if (max_seq_len < 0 || k_max < 0 || (!k_per_seq && k_uniform < 0)) return HA_ERR_INVALID_ARG;
    if (((uintptr_t)k_codes & 15) || (kc_stride_b & 3) || (kc_stride_h & 3)) return HA_ERR_INVALID_ARG;
    if ((long long)shape->n_sink + shape->n_local > k_max) return HA_ERR_INVALID_ARG;   // idx rows must hold the windows
    return HA_OK;
}

int ha_score_topk(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes, int64_t kc_stride_b,
                  int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                  int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h,
                  int32_t *count, int32_t *hist_out, void *workspace, size_t ws_bytes, void *stream) {
    HA_TRY(check_score_args(shape, q_codes, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_uniform, k_per_seq,
                            max_seq_len, k_max, idx, count));
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, max_seq_len, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    HA_CUDA(launch_score_topk(shape->batch, shape->n_q_heads, shape->n_kv_heads, q_codes, k_codes, kc_stride_b,
                              kc_stride_h, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx, idx_stride_b,
                              idx_stride_h, count, hist_out, ws_ptr<int32_t>(workspace, L.off_hist),
                              ws_ptr<unsigned char>(workspace, L.off_scores), (cudaStream_t)stream,
                              Windows{shape->n_sink, shape->n_local}));
    return HA_OK;
}

int ha_score_topk_sum(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes, int64_t kc_stride_b,
                      int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                      int32_t k_max, int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                      int32_t *hist_out, void *stream) {
    HA_TRY(check_score_args(shape, q_codes, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_uniform, k_per_seq, 0, k_max,
                            idx, count));
    if (shape->batch == 0) return HA_OK;
    HA_CUDA(launch_score_topk_sum(shape->batch, shape->n_q_heads, shape->n_kv_heads, q_codes, k_codes, kc_stride_b,
                                  kc_stride_h, seq_lens, k_per_seq, k_uniform, k_max, idx, idx_stride_b, idx_stride_h,
                                  count, hist_out, (cudaStream_t)stream, Windows{shape->n_sink, shape->n_local}));
    return HA_OK;
}

int ha_gather_attn(const ha_shape *shape, const uint16_t *q, const ha_tensor *K, const ha_tensor *V,
                   const int32_t *seq_lens, const int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h,
                   const int32_t *count, int32_t k_max, uint16_t *out, float *lse, void *workspace, size_t ws_bytes,
                   void *stream) {
    HA_TRY(check_shape(shape));
    HA_TRY(check_tensor(K));
    HA_TRY(check_tensor(V));
    if (!q || !seq_lens || !idx || !count || !out || k_max < 0) return HA_ERR_INVALID_ARG;
    if ((uintptr_t)q & 15) return HA_ERR_INVALID_ARG;
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, -1, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    if (gather_cluster_eligible(shape->batch, shape->n_q_heads, shape->n_kv_heads, k_max)) {
        // few units, short lists: one cluster per unit, merged through distributed shared memory
        HA_CUDA(launch_gather_cluster(shape->batch, shape->n_q_heads, shape->n_kv_heads, shape->sm_scale, q, view(K), view(V),
                                      seq_lens, idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                                      ws_ptr<uint32_t>(workspace, 0), (cudaStream_t)stream));
        return HA_OK;
    }
    HA_CUDA(launch_attention(true, shape->batch, shape->n_q_heads, shape->n_kv_heads, shape->sm_scale, q, view(K),
                             view(V), seq_lens, idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                             ws_ptr<float>(workspace, L.off_part_ml), ws_ptr<float>(workspace, L.off_part_acc),
                             ws_ptr<int32_t>(workspace, L.off_tickets), ws_ptr<uint32_t>(workspace, 0),
                             (cudaStream_t)stream));
    return HA_OK;
}

// ---- one list per QUERY head: no reduction over the group (the third reading of how a group selects)

int ha_score_topk_per_head(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *k_codes, int64_t kc_stride_b,
                           int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                           int32_t k_max, int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count,
                           int32_t *hist_out, void *stream) {
    HA_TRY(check_score_args(shape, q_codes, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_uniform, k_per_seq, 0, k_max,
                            idx, count));
    if ((long long)shape->n_q_heads * shape->batch > kMaxUnits) return HA_ERR_UNSUPPORTED;
    if (shape->batch == 0) return HA_OK;
    HA_CUDA(launch_score_topk_sum(shape->batch, shape->n_q_heads, shape->n_kv_heads, q_codes, k_codes, kc_stride_b,
                                  kc_stride_h, seq_lens, k_per_seq, k_uniform, k_max, idx, idx_stride_b, idx_stride_h,
                                  count, hist_out, (cudaStream_t)stream, Windows{shape->n_sink, shape->n_local}, true));
    return HA_OK;
}

int ha_gather_attn_per_head(const ha_shape *shape, const uint16_t *q, const ha_tensor *K, const ha_tensor *V,
                            const int32_t *seq_lens, const int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h,
                            const int32_t *count, int32_t k_max, uint16_t *out, float *lse, void *workspace,
                            size_t ws_bytes, void *stream) {
    HA_TRY(check_shape(shape));
    HA_TRY(check_tensor(K));
    HA_TRY(check_tensor(V));
    if (!q || !seq_lens || !idx || !count || !out || k_max < 0) return HA_ERR_INVALID_ARG;
    if ((uintptr_t)q & 15) return HA_ERR_INVALID_ARG;
    ha_shape units = *shape;             // every query head is a unit: the scratch is laid out for that many
    units.n_kv_heads = shape->n_q_heads;
    HA_TRY(check_shape(&units));
    WorkspaceLayout L;
    HA_TRY(check_workspace(&units, -1, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    int shift = 0;
    while ((shape->n_kv_heads << shift) < shape->n_q_heads) ++shift;
    HA_CUDA(launch_attention(true, shape->batch, shape->n_q_heads, shape->n_q_heads, shape->sm_scale, q, view(K), view(V),
                             seq_lens, idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                             ws_ptr<float>(workspace, L.off_part_ml), ws_ptr<float>(workspace, L.off_part_acc),
                             ws_ptr<int32_t>(workspace, L.off_tickets), ws_ptr<uint32_t>(workspace, 0),
                             (cudaStream_t)stream, 0, nullptr, 0, Windows{0, 0}, nullptr, 0, 0, shift));
    return HA_OK;
}

int ha_gather_attn_paged(const ha_shape *shape, const uint16_t *q, const ha_tensor *K_pool, const ha_tensor *V_pool,
                         const int32_t *block_table, int64_t bt_stride_b, int32_t page_size, const int32_t *seq_lens,
                         const int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, const int32_t *count,
                         int32_t k_max, uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream) {
    HA_TRY(check_shape(shape));
    HA_TRY(check_tensor(K_pool));
    HA_TRY(check_tensor(V_pool));
    if (!q || !block_table || !seq_lens || !idx || !count || !out || k_max < 0) return HA_ERR_INVALID_ARG;
    if ((uintptr_t)q & 15) return HA_ERR_INVALID_ARG;
    if (page_size <= 0 || (page_size & (page_size - 1)) || page_size > 65536) return HA_ERR_INVALID_ARG;
    // a page is page_size consecutive slots: both pools must step through pages in whole rows, the same way
    if (K_pool->stride_b % K_pool->stride_n != 0 || V_pool->stride_b % V_pool->stride_n != 0 ||
        K_pool->stride_b / K_pool->stride_n != V_pool->stride_b / V_pool->stride_n)
        return HA_ERR_INVALID_ARG;
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, -1, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    int shift = 0;
    while ((1 << shift) < page_size) ++shift;
    if (gather_cluster_eligible(shape->batch, shape->n_q_heads, shape->n_kv_heads, k_max)) {
        HA_CUDA(launch_gather_cluster(shape->batch, shape->n_q_heads, shape->n_kv_heads, shape->sm_scale, q, view(K_pool),
                                      view(V_pool), seq_lens, idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                                      ws_ptr<uint32_t>(workspace, 0), (cudaStream_t)stream, block_table, bt_stride_b, shift));
        return HA_OK;
    }
    HA_CUDA(launch_attention(true, shape->batch, shape->n_q_heads, shape->n_kv_heads, shape->sm_scale, q, view(K_pool),
                             view(V_pool), seq_lens, idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                             ws_ptr<float>(workspace, L.off_part_ml), ws_ptr<float>(workspace, L.off_part_acc),
                             ws_ptr<int32_t>(workspace, L.off_tickets), ws_ptr<uint32_t>(workspace, 0),
                             (cudaStream_t)stream, 0, nullptr, 0, Windows{0, 0}, block_table, bt_stride_b, shift));
    return HA_OK;
}

int ha_dense_decode(const ha_shape *shape, const uint16_t *q, const ha_tensor *K, const ha_tensor *V,
                    const int32_t *seq_lens, int32_t max_seq_len, uint16_t *out, float *lse, void *workspace,
                    size_t ws_bytes, void *stream) {
    HA_TRY(check_shape(shape));
    HA_TRY(check_tensor(K));
    HA_TRY(check_tensor(V));
    if (!q || !seq_lens || !out || max_seq_len < 0) return HA_ERR_INVALID_ARG;
    if ((uintptr_t)q & 15) return HA_ERR_INVALID_ARG;
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, -1, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    HA_CUDA(launch_attention(false, shape->batch, shape->n_q_heads, shape->n_kv_heads, shape->sm_scale, q, view(K),
                             view(V), seq_lens, nullptr, 0, 0, nullptr, max_seq_len, out, lse,
                             ws_ptr<float>(workspace, L.off_part_ml), ws_ptr<float>(workspace, L.off_part_acc),
                             ws_ptr<int32_t>(workspace, L.off_tickets), ws_ptr<uint32_t>(workspace, 0),
                             (cudaStream_t)stream));
    return HA_OK;
}

static int sparse_decode_impl(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k, const uint16_t *q,
                              const uint16_t *k_new, const ha_tensor *K, const ha_tensor *V, const int32_t *block_table,
                              int64_t bt_stride_b, int page_shift, uint32_t *k_codes, int64_t kc_stride_b,
                              int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                              int32_t max_seq_len, int32_t k_max, uint32_t *q_codes, int32_t *idx, int64_t idx_stride_b,
                              int64_t idx_stride_h, int32_t *count, uint16_t *out, float *lse, void *workspace,
                              size_t ws_bytes, void *stream, const uint16_t *v_new_host = nullptr, bool pipelined = false,
                              CodePages code_pages = CodePages{nullptr, 0, 0, 0, 0}) {
    HA_TRY(check_score_args(shape, q_codes, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_uniform, k_per_seq,
                            max_seq_len, k_max, idx, count));
    HA_TRY(check_mapping(map_q, shape->n_kv_heads));
    if (k_new) HA_TRY(check_mapping(map_k, shape->n_kv_heads));
    const bool codes_paged = code_pages.table != nullptr;   // then only the kernel-by-kernel path knows the layout
    if (codes_paged && (pipelined || v_new_host)) return HA_ERR_UNSUPPORTED;
    HA_TRY(check_tensor(K));
    HA_TRY(check_tensor(V));
    if (!q || !out || ((uintptr_t)q & 15)) return HA_ERR_INVALID_ARG;
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, max_seq_len, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const int B = shape->batch, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads;

    if (pipelined && !pipe_step_eligible(B, Hq, Hkv)) return HA_ERR_UNSUPPORTED;
    if (!pipelined && !codes_paged && fused_step_eligible(B, Hq, Hkv, max_seq_len, k_max)) {
        // small batch: the whole step is one cluster kernel
        HA_CUDA(launch_fused_step(B, Hq, Hkv, shape->sm_scale, view(map_q), k_new ? view(map_k) : MapView{}, q, k_new,
                                  view(K), view(V), k_codes, kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform,
                                  max_seq_len, k_max, q_codes, idx, idx_stride_b, idx_stride_h, count, out, lse, st,
                                  Windows{shape->n_sink, shape->n_local}, block_table, bt_stride_b, page_shift, v_new_host));
        return HA_OK;
    }
    if (v_new_host) return HA_ERR_INVALID_ARG;   // only the fused kernel appends by itself

    EncodeJob jq{};
    jq.x = q; jq.x_sb = (long long)Hq * kD; jq.x_sh = kD;
    jq.codes = q_codes; jq.c_sb = Hq; jq.c_sh = 1;
    jq.slot = nullptr; jq.slot_minus_one = 0;
    jq.n_heads = Hq; jq.heads_per_kv = Hq / Hkv; jq.n_cta = B * Hkv;
    jq.map = view(map_q);
    EncodeJob jk{};
    if (k_new) {
        jk.x = k_new; jk.x_sb = (long long)Hkv * kD; jk.x_sh = kD;
        jk.codes = k_codes; jk.c_sb = kc_stride_b; jk.c_sh = kc_stride_h;
        jk.slot = seq_lens; jk.slot_minus_one = 1;
        jk.n_heads = Hkv; jk.heads_per_kv = 1; jk.n_cta = B * Hkv;
        jk.map = view(map_k);
        jk.pages = code_pages;
    }
    HA_CUDA(launch_encode_vectors(jq, jk, st));
    if (pipelined) {
        // SCORE + TOPK and GATHER-ATT in one persistent kernel: the scoring of later units runs under the row fetch of earlier ones
        int32_t *counters = ws_ptr<int32_t>(workspace, L.off_tickets);
        const size_t units = (size_t)B * Hkv;
        HA_CUDA(launch_pipe_step(B, Hq, Hkv, shape->sm_scale, q_codes, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_per_seq,
                                 k_uniform, max_seq_len, k_max, idx, idx_stride_b, idx_stride_h, count, q, view(K), view(V), out,
                                 lse, counters, counters + units, counters + 2 * units, ws_ptr<int32_t>(workspace, L.off_hist),
                                 ws_ptr<unsigned char>(workspace, L.off_scores), (long long)score_row_bytes(max_seq_len),
                                 ws_ptr<float>(workspace, L.off_part_ml), ws_ptr<float>(workspace, L.off_part_acc),
                                 ws_ptr<uint32_t>(workspace, 0), st, Windows{shape->n_sink, shape->n_local}, block_table,
                                 bt_stride_b, page_shift));
        return HA_OK;
    }
    HA_CUDA(launch_score_topk(B, Hq, Hkv, q_codes, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform,
                              max_seq_len, k_max, idx, idx_stride_b, idx_stride_h, count, nullptr,
                              ws_ptr<int32_t>(workspace, L.off_hist), ws_ptr<unsigned char>(workspace, L.off_scores), st,
                              Windows{shape->n_sink, shape->n_local}, code_pages));
    if (gather_cluster_eligible(B, Hq, Hkv, k_max)) {
        // up to a cluster per unit resident at once and short lists: GATHER-ATT with the states merged in shared memory
        HA_CUDA(launch_gather_cluster(B, Hq, Hkv, shape->sm_scale, q, view(K), view(V), seq_lens, idx, idx_stride_b,
                                      idx_stride_h, count, k_max, out, lse, ws_ptr<uint32_t>(workspace, 0), st, block_table,
                                      bt_stride_b, page_shift));
        return HA_OK;
    }
    HA_CUDA(launch_attention(true, B, Hq, Hkv, shape->sm_scale, q, view(K), view(V), seq_lens, idx, idx_stride_b,
                             idx_stride_h, count, k_max, out, lse, ws_ptr<float>(workspace, L.off_part_ml),
                             ws_ptr<float>(workspace, L.off_part_acc), ws_ptr<int32_t>(workspace, L.off_tickets),
                             ws_ptr<uint32_t>(workspace, 0), st, /*count_from_k=*/1, k_per_seq, k_uniform,
                             Windows{shape->n_sink, shape->n_local}, block_table, bt_stride_b, page_shift));
    return HA_OK;
}

int ha_sparse_decode(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k, const uint16_t *q,
                     const uint16_t *k_new, const ha_tensor *K, const ha_tensor *V, uint32_t *k_codes,
                     int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                     int32_t k_uniform, int32_t max_seq_len, int32_t k_max, uint32_t *q_codes, int32_t *idx,
                     int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, uint16_t *out, float *lse,
                     void *workspace, size_t ws_bytes, void *stream) {
    return sparse_decode_impl(shape, map_q, map_k, q, k_new, K, V, nullptr, 0, 0, k_codes, kc_stride_b, kc_stride_h, seq_lens,
                              k_per_seq, k_uniform, max_seq_len, k_max, q_codes, idx, idx_stride_b, idx_stride_h, count, out,
                              lse, workspace, ws_bytes, stream);
}

int ha_sparse_decode_pipelined(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k, const uint16_t *q,
                               const uint16_t *k_new, const ha_tensor *K, const ha_tensor *V, uint32_t *k_codes,
                               int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                               int32_t k_uniform, int32_t max_seq_len, int32_t k_max, uint32_t *q_codes, int32_t *idx,
                               int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, uint16_t *out, float *lse,
                               void *workspace, size_t ws_bytes, void *stream) {
    return sparse_decode_impl(shape, map_q, map_k, q, k_new, K, V, nullptr, 0, 0, k_codes, kc_stride_b, kc_stride_h, seq_lens,
                              k_per_seq, k_uniform, max_seq_len, k_max, q_codes, idx, idx_stride_b, idx_stride_h, count, out,
                              lse, workspace, ws_bytes, stream, nullptr, /*pipelined=*/true);
}

int ha_sparse_decode_paged(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k, const uint16_t *q,
                           const uint16_t *k_new, const ha_tensor *K_pool, const ha_tensor *V_pool,
                           const int32_t *block_table, int64_t bt_stride_b, int32_t page_size, uint32_t *k_codes,
                           int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                           int32_t k_uniform, int32_t max_seq_len, int32_t k_max, uint32_t *q_codes, int32_t *idx,
                           int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, uint16_t *out, float *lse,
                           void *workspace, size_t ws_bytes, void *stream) {
    if (!block_table || !K_pool || !V_pool) return HA_ERR_INVALID_ARG;
    if (page_size <= 0 || (page_size & (page_size - 1)) || page_size > 65536) return HA_ERR_INVALID_ARG;
    if (K_pool->stride_n <= 0 || V_pool->stride_n <= 0 || K_pool->stride_b % K_pool->stride_n != 0 ||
        V_pool->stride_b % V_pool->stride_n != 0 || K_pool->stride_b / K_pool->stride_n != V_pool->stride_b / V_pool->stride_n)
        return HA_ERR_INVALID_ARG;
    int shift = 0;
    while ((1 << shift) < page_size) ++shift;
    return sparse_decode_impl(shape, map_q, map_k, q, k_new, K_pool, V_pool, block_table, bt_stride_b, shift, k_codes,
                              kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, q_codes, idx,
                              idx_stride_b, idx_stride_h, count, out, lse, workspace, ws_bytes, stream);
}

// ---- paged signature cache: the signatures live in a pool beside the K/V pools, addressed by the same block table

static int check_code_pool(const uint32_t *code_pool, int64_t cp_stride_page, int64_t cp_stride_head, const int32_t *block_table,
                           int32_t page_size, CodePages *cp, int64_t bt_stride_b) {
    if (!code_pool || !block_table) return HA_ERR_INVALID_ARG;
    if (page_size <= 0 || (page_size & (page_size - 1)) || page_size > 65536) return HA_ERR_INVALID_ARG;
    // pages of four tokens or more are read sixteen bytes at a time
    if (((uintptr_t)code_pool & 15) || (page_size >= 4 && ((cp_stride_page & 3) || (cp_stride_head & 3)))) return HA_ERR_INVALID_ARG;
    int shift = 0;
    while ((1 << shift) < page_size) ++shift;
    *cp = CodePages{block_table, (long long)bt_stride_b, (long long)cp_stride_page, (long long)cp_stride_head, shift};
    return HA_OK;
}

int ha_score_topk_paged(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *code_pool, int64_t cp_stride_page,
                        int64_t cp_stride_head, const int32_t *block_table, int64_t bt_stride_b, int32_t page_size,
                        const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform, int32_t max_seq_len, int32_t k_max,
                        int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, int32_t *hist_out,
                        void *workspace, size_t ws_bytes, void *stream) {
    CodePages cp;
    HA_TRY(check_code_pool(code_pool, cp_stride_page, cp_stride_head, block_table, page_size, &cp, bt_stride_b));
    HA_TRY(check_score_args(shape, q_codes, code_pool, 0, 0, seq_lens, k_uniform, k_per_seq, max_seq_len, k_max, idx, count));
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, max_seq_len, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    HA_CUDA(launch_score_topk(shape->batch, shape->n_q_heads, shape->n_kv_heads, q_codes, code_pool, 0, 0, seq_lens, k_per_seq,
                              k_uniform, max_seq_len, k_max, idx, idx_stride_b, idx_stride_h, count, hist_out,
                              ws_ptr<int32_t>(workspace, L.off_hist), ws_ptr<unsigned char>(workspace, L.off_scores),
                              (cudaStream_t)stream, Windows{shape->n_sink, shape->n_local}, cp));
    return HA_OK;
}

int ha_score_topk_per_head_paged(const ha_shape *shape, const uint32_t *q_codes, const uint32_t *code_pool,
                                 int64_t cp_stride_page, int64_t cp_stride_head, const int32_t *block_table,
                                 int64_t bt_stride_b, int32_t page_size, const int32_t *seq_lens, const int32_t *k_per_seq,
                                 int32_t k_uniform, int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                                 int64_t idx_stride_h, int32_t *count, int32_t *hist_out, void *workspace, size_t ws_bytes,
                                 void *stream) {
    CodePages cp;
    HA_TRY(check_code_pool(code_pool, cp_stride_page, cp_stride_head, block_table, page_size, &cp, bt_stride_b));
    HA_TRY(check_score_args(shape, q_codes, code_pool, 0, 0, seq_lens, k_uniform, k_per_seq, max_seq_len, k_max, idx, count));
    ha_shape units = *shape;             // every query head is a unit: the scratch is laid out for that many
    units.n_kv_heads = shape->n_q_heads;
    HA_TRY(check_shape(&units));
    WorkspaceLayout L;
    HA_TRY(check_workspace(&units, max_seq_len, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    int shift = 0;
    while ((shape->n_kv_heads << shift) < shape->n_q_heads) ++shift;
    HA_CUDA(launch_score_topk(shape->batch, shape->n_q_heads, shape->n_kv_heads, q_codes, code_pool, 0, 0, seq_lens, k_per_seq,
                              k_uniform, max_seq_len, k_max, idx, idx_stride_b, idx_stride_h, count, hist_out,
                              ws_ptr<int32_t>(workspace, L.off_hist), ws_ptr<unsigned char>(workspace, L.off_scores),
                              (cudaStream_t)stream, Windows{shape->n_sink, shape->n_local}, cp, shift));
    return HA_OK;
}

int ha_gather_attn_per_head_paged(const ha_shape *shape, const uint16_t *q, const ha_tensor *K_pool, const ha_tensor *V_pool,
                                  const int32_t *block_table, int64_t bt_stride_b, int32_t page_size, const int32_t *seq_lens,
                                  const int32_t *idx, int64_t idx_stride_b, int64_t idx_stride_h, const int32_t *count,
                                  int32_t k_max, uint16_t *out, float *lse, void *workspace, size_t ws_bytes, void *stream) {
    HA_TRY(check_shape(shape));
    HA_TRY(check_tensor(K_pool));
    HA_TRY(check_tensor(V_pool));
    if (!q || !block_table || !seq_lens || !idx || !count || !out || k_max < 0 || ((uintptr_t)q & 15)) return HA_ERR_INVALID_ARG;
    if (page_size <= 0 || (page_size & (page_size - 1)) || page_size > 65536) return HA_ERR_INVALID_ARG;
    if (K_pool->stride_b % K_pool->stride_n != 0 || V_pool->stride_b % V_pool->stride_n != 0 ||
        K_pool->stride_b / K_pool->stride_n != V_pool->stride_b / V_pool->stride_n)
        return HA_ERR_INVALID_ARG;
    ha_shape units = *shape;
    units.n_kv_heads = shape->n_q_heads;
    HA_TRY(check_shape(&units));
    WorkspaceLayout L;
    HA_TRY(check_workspace(&units, -1, workspace, ws_bytes, &L));
    if (shape->batch == 0) return HA_OK;
    int kv_shift = 0, page_shift = 0;
    while ((shape->n_kv_heads << kv_shift) < shape->n_q_heads) ++kv_shift;
    while ((1 << page_shift) < page_size) ++page_shift;
    HA_CUDA(launch_attention(true, shape->batch, shape->n_q_heads, shape->n_q_heads, shape->sm_scale, q, view(K_pool), view(V_pool),
                             seq_lens, idx, idx_stride_b, idx_stride_h, count, k_max, out, lse,
                             ws_ptr<float>(workspace, L.off_part_ml), ws_ptr<float>(workspace, L.off_part_acc),
                             ws_ptr<int32_t>(workspace, L.off_tickets), ws_ptr<uint32_t>(workspace, 0), (cudaStream_t)stream, 0,
                             nullptr, 0, Windows{0, 0}, block_table, bt_stride_b, page_shift, kv_shift));
    return HA_OK;
}

int ha_encode_append_paged(const ha_mapping *map, const uint16_t *k_new, int32_t batch, uint32_t *code_pool,
                           int64_t cp_stride_page, int64_t cp_stride_head, const int32_t *block_table, int64_t bt_stride_b,
                           int32_t page_size, const int32_t *seq_lens, void *stream) {
    HA_TRY(check_mapping(map, 0));
    CodePages cp;
    HA_TRY(check_code_pool(code_pool, cp_stride_page, cp_stride_head, block_table, page_size, &cp, bt_stride_b));
    if (!k_new || ((uintptr_t)k_new & 15) || !seq_lens || batch < 0 || batch > 65535) return HA_ERR_INVALID_ARG;
    if (batch == 0) return HA_OK;
    const int Hkv = map->n_kv_heads;
    EncodeJob jk{};
    jk.x = k_new; jk.x_sb = (long long)Hkv * kD; jk.x_sh = kD;
    jk.codes = code_pool; jk.slot = seq_lens; jk.slot_minus_one = 1;
    jk.n_heads = Hkv; jk.heads_per_kv = 1; jk.n_cta = batch * Hkv;
    jk.map = view(map);
    jk.pages = cp;
    EncodeJob none{};
    HA_CUDA(launch_encode_vectors(jk, none, (cudaStream_t)stream));
    return HA_OK;
}

int ha_sparse_decode_paged_codes(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k, const uint16_t *q,
                                 const uint16_t *k_new, const ha_tensor *K_pool, const ha_tensor *V_pool, uint32_t *code_pool,
                                 int64_t cp_stride_page, int64_t cp_stride_head, const int32_t *block_table, int64_t bt_stride_b,
                                 int32_t page_size, const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                                 int32_t max_seq_len, int32_t k_max, uint32_t *q_codes, int32_t *idx, int64_t idx_stride_b,
                                 int64_t idx_stride_h, int32_t *count, uint16_t *out, float *lse, void *workspace,
                                 size_t ws_bytes, void *stream) {
    if (!K_pool || !V_pool) return HA_ERR_INVALID_ARG;
    CodePages cp;
    HA_TRY(check_code_pool(code_pool, cp_stride_page, cp_stride_head, block_table, page_size, &cp, bt_stride_b));
    if (K_pool->stride_n <= 0 || V_pool->stride_n <= 0 || K_pool->stride_b % K_pool->stride_n != 0 ||
        V_pool->stride_b % V_pool->stride_n != 0 || K_pool->stride_b / K_pool->stride_n != V_pool->stride_b / V_pool->stride_n)
        return HA_ERR_INVALID_ARG;
    return sparse_decode_impl(shape, map_q, map_k, q, k_new, K_pool, V_pool, block_table, bt_stride_b, cp.shift, code_pool, 0, 0,
                              seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, q_codes, idx, idx_stride_b, idx_stride_h, count,
                              out, lse, workspace, ws_bytes, stream, nullptr, false, cp);
}

// Both host-buffer entries: block_table == NULL is the contiguous cache, else K / V are pools (page_shift = log2 of
// the page size).
static int sparse_decode_host_impl(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                                   const uint16_t *q_host, const uint16_t *k_new_host, const uint16_t *v_new_host,
                                   const ha_tensor *K, const ha_tensor *V, const int32_t *block_table, int64_t bt_stride_b,
                                   int page_shift, uint32_t *k_codes, int64_t kc_stride_b, int64_t kc_stride_h,
                                   const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                                   int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                                   int64_t idx_stride_h, int32_t *count, uint16_t *out_host, void *workspace,
                                   size_t ws_bytes, void *stream) {
    HA_TRY(check_shape(shape));
    if (!q_host || !k_new_host || !v_new_host || !out_host) return HA_ERR_INVALID_ARG;
    HA_TRY(check_tensor(K));
    HA_TRY(check_tensor(V));
    HA_TRY(check_mapping(map_q, shape->n_kv_heads));
    HA_TRY(check_mapping(map_k, shape->n_kv_heads));
    WorkspaceLayout L;
    HA_TRY(check_workspace(shape, max_seq_len, workspace, ws_bytes, &L));
    HA_TRY(check_score_args(shape, ws_ptr<uint32_t>(workspace, L.off_qcodes), k_codes, kc_stride_b, kc_stride_h,
                            seq_lens, k_uniform, k_per_seq, max_seq_len, k_max, idx, count));
    if (shape->batch == 0) return HA_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const int B = shape->batch, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads;
    uint16_t *dq = ws_ptr<uint16_t>(workspace, L.off_stage_q);
    uint16_t *dk = ws_ptr<uint16_t>(workspace, L.off_stage_k);
    uint16_t *dv = ws_ptr<uint16_t>(workspace, L.off_stage_v);
    uint16_t *dout = ws_ptr<uint16_t>(workspace, L.off_stage_out);
    uint32_t *dqc = ws_ptr<uint32_t>(workspace, L.off_qcodes);
    // Pinned host buffers that the device can address (cudaHostAlloc / cudaHostRegister under unified
    // addressing) are read and written by the kernels themselves: one small kernel pulls q, k_new and
    // v_new across the bus and the last kernel of the step writes `out` straight into host memory.
    // Anything else goes through staged copies.
    auto mapped = [](const void *p) -> void * {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return (at.type == cudaMemoryTypeHost) ? at.devicePointer : nullptr;
    };
    const uint16_t *mq = reinterpret_cast<const uint16_t *>(mapped(q_host));
    const uint16_t *mkn = reinterpret_cast<const uint16_t *>(mapped(k_new_host));
    const uint16_t *mvn = reinterpret_cast<const uint16_t *>(mapped(v_new_host));
    uint16_t *mout = reinterpret_cast<uint16_t *>(mapped(out_host));
    if (!block_table && mq && mkn && mvn && mout && fused_step_from_host_eligible(B, Hq, Hkv, max_seq_len, k_max)) {
        // one launch: the fused kernel reads q / k_new / v_new across the bus, appends the new rows and writes `out`
        HA_TRY(sparse_decode_impl(shape, map_q, map_k, mq, mkn, K, V, nullptr, 0, 0, k_codes, kc_stride_b, kc_stride_h,
                                  seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, dqc, idx, idx_stride_b, idx_stride_h,
                                  count, mout, nullptr, workspace, ws_bytes, stream, mvn));
    } else if (mq && mkn && mvn && mout) {
        HA_CUDA(launch_append_kv(B, Hq, Hkv, mkn, mvn, view(K), view(V), seq_lens, mq, dq, dk, st, block_table, bt_stride_b,
                                 page_shift));
        HA_TRY(sparse_decode_impl(shape, map_q, map_k, dq, dk, K, V, block_table, bt_stride_b, page_shift, k_codes,
                                  kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, dqc, idx,
                                  idx_stride_b, idx_stride_h, count, mout, nullptr, workspace, ws_bytes, stream));
    } else {
        HA_CUDA(cudaMemcpyAsync(dq, q_host, (size_t)B * Hq * kD * 2, cudaMemcpyHostToDevice, st));
        HA_CUDA(cudaMemcpyAsync(dk, k_new_host, (size_t)B * Hkv * kD * 2, cudaMemcpyHostToDevice, st));
        HA_CUDA(cudaMemcpyAsync(dv, v_new_host, (size_t)B * Hkv * kD * 2, cudaMemcpyHostToDevice, st));
        HA_CUDA(launch_append_kv(B, Hq, Hkv, dk, dv, view(K), view(V), seq_lens, nullptr, nullptr, nullptr, st, block_table,
                                 bt_stride_b, page_shift));
        HA_TRY(sparse_decode_impl(shape, map_q, map_k, dq, dk, K, V, block_table, bt_stride_b, page_shift, k_codes,
                                  kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, dqc, idx,
                                  idx_stride_b, idx_stride_h, count, dout, nullptr, workspace, ws_bytes, stream));
        HA_CUDA(cudaMemcpyAsync(out_host, dout, (size_t)B * Hq * kD * 2, cudaMemcpyDeviceToHost, st));
    }
    HA_CUDA(cudaStreamSynchronize(st));
    return HA_OK;
}

int ha_sparse_decode_host(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                          const uint16_t *q_host, const uint16_t *k_new_host, const uint16_t *v_new_host,
                          const ha_tensor *K, const ha_tensor *V, uint32_t *k_codes, int64_t kc_stride_b,
                          int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq, int32_t k_uniform,
                          int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                          int64_t idx_stride_h, int32_t *count, uint16_t *out_host, void *workspace, size_t ws_bytes,
                          void *stream) {
    return sparse_decode_host_impl(shape, map_q, map_k, q_host, k_new_host, v_new_host, K, V, nullptr, 0, 0, k_codes,
                                   kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx,
                                   idx_stride_b, idx_stride_h, count, out_host, workspace, ws_bytes, stream);
}

int ha_sparse_decode_paged_host(const ha_shape *shape, const ha_mapping *map_q, const ha_mapping *map_k,
                                const uint16_t *q_host, const uint16_t *k_new_host, const uint16_t *v_new_host,
                                const ha_tensor *K_pool, const ha_tensor *V_pool, const int32_t *block_table,
                                int64_t bt_stride_b, int32_t page_size, uint32_t *k_codes, int64_t kc_stride_b,
                                int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                                int32_t k_uniform, int32_t max_seq_len, int32_t k_max, int32_t *idx,
                                int64_t idx_stride_b, int64_t idx_stride_h, int32_t *count, uint16_t *out_host,
                                void *workspace, size_t ws_bytes, void *stream) {
    if (!block_table || !K_pool || !V_pool) return HA_ERR_INVALID_ARG;
    if (page_size <= 0 || (page_size & (page_size - 1)) || page_size > 65536) return HA_ERR_INVALID_ARG;
    if (K_pool->stride_n <= 0 || V_pool->stride_n <= 0 || K_pool->stride_b % K_pool->stride_n != 0 ||
        V_pool->stride_b % V_pool->stride_n != 0 || K_pool->stride_b / K_pool->stride_n != V_pool->stride_b / V_pool->stride_n)
        return HA_ERR_INVALID_ARG;
    int shift = 0;
    while ((1 << shift) < page_size) ++shift;
    return sparse_decode_host_impl(shape, map_q, map_k, q_host, k_new_host, v_new_host, K_pool, V_pool, block_table,
                                   bt_stride_b, shift, k_codes, kc_stride_b, kc_stride_h, seq_lens, k_per_seq, k_uniform,
                                   max_seq_len, k_max, idx, idx_stride_b, idx_stride_h, count, out_host, workspace,
                                   ws_bytes, stream);
}

int ha_score_wide(const uint64_t *q_code, const uint64_t *k_codes, int64_t n, int32_t n_bits, uint16_t *scores,
                  void *stream) {
    if (n < 0 || !q_code || (n > 0 && (!k_codes || !scores))) return HA_ERR_INVALID_ARG;
    if (n_bits != 64 && n_bits != 128 && n_bits != 256 && n_bits != 512) return HA_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(k_codes) & 15) || (reinterpret_cast<uintptr_t>(scores) & 3) ||
        (reinterpret_cast<uintptr_t>(q_code) & 7))
        return HA_ERR_INVALID_ARG;
    HA_CUDA(launch_score_wide(q_code, k_codes, n, n_bits / 64, scores, (cudaStream_t)stream));
    return HA_OK;
}

static bool wide_bits_ok(int32_t n_bits) { return n_bits == 64 || n_bits == 128 || n_bits == 256 || n_bits == 512; }

int ha_encode_wide(const ha_mapping *map, int32_t heads_per_kv, const ha_tensor *x, int32_t batch, int32_t n_heads,
                   int32_t n_tokens, uint64_t *codes, int64_t c_stride_b, int64_t c_stride_h, const int32_t *slot,
                   void *stream) {
    if (!map || !map->w1 || !map->w2 || !map->w3) return HA_ERR_INVALID_ARG;
    if (map->in_dim != kD || map->hid_dim != kHid || !wide_bits_ok(map->n_bits)) return HA_ERR_UNSUPPORTED;
    if (map->n_kv_heads <= 0 || (((uintptr_t)map->w1 | (uintptr_t)map->w2 | (uintptr_t)map->w3) & 15)) return HA_ERR_INVALID_ARG;
    HA_TRY(check_tensor(x));
    if (!codes || ((uintptr_t)codes & 7) || batch < 0 || n_heads <= 0 || n_tokens < 0 || heads_per_kv <= 0) return HA_ERR_INVALID_ARG;
    if (n_heads % heads_per_kv != 0 || n_heads / heads_per_kv != map->n_kv_heads) return HA_ERR_INVALID_ARG;
    if (slot && n_tokens != 1) return HA_ERR_INVALID_ARG;
    if (batch > 65535 || n_heads > 65535) return HA_ERR_UNSUPPORTED;
    if (batch == 0 || n_tokens == 0) return HA_OK;
    HA_CUDA(launch_encode_wide(view(map), map->n_bits, heads_per_kv, view(x), batch, n_heads, n_tokens, codes, c_stride_b,
                               c_stride_h, slot, (cudaStream_t)stream));
    return HA_OK;
}

size_t ha_workspace_bytes_wide(const ha_shape *shape, int32_t max_seq_len) {
    if (check_shape(shape) != HA_OK || max_seq_len < 0) return 0;
    return wide_workspace_bytes(shape->batch, shape->n_kv_heads, max_seq_len);
}

int ha_score_topk_wide(const ha_shape *shape, int32_t n_bits, const uint64_t *q_codes, const uint64_t *k_codes,
                       int64_t kc_stride_b, int64_t kc_stride_h, const int32_t *seq_lens, const int32_t *k_per_seq,
                       int32_t k_uniform, int32_t max_seq_len, int32_t k_max, int32_t *idx, int64_t idx_stride_b,
                       int64_t idx_stride_h, int32_t *count, int32_t *hist_out, void *workspace, size_t ws_bytes,
                       void *stream) {
    HA_TRY(check_shape(shape));
    if (!wide_bits_ok(n_bits)) return HA_ERR_UNSUPPORTED;
    if (!q_codes || !k_codes || !seq_lens || !idx || !count) return HA_ERR_INVALID_ARG;
    if (max_seq_len < 0 || k_max < 0 || (!k_per_seq && k_uniform < 0)) return HA_ERR_INVALID_ARG;
    if (((uintptr_t)k_codes & 15) || ((uintptr_t)q_codes & 7)) return HA_ERR_INVALID_ARG;
    if (n_bits > 64 && ((kc_stride_b & 1) || (kc_stride_h & 1))) return HA_ERR_INVALID_ARG;   // 16-byte loads
    if ((long long)shape->n_sink + shape->n_local > k_max) return HA_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return HA_ERR_WORKSPACE;
    if (ws_bytes < wide_workspace_bytes(shape->batch, shape->n_kv_heads, max_seq_len)) return HA_ERR_WORKSPACE;
    if (shape->batch == 0) return HA_OK;
    HA_CUDA(launch_score_topk_wide(shape->batch, shape->n_q_heads, shape->n_kv_heads, n_bits, q_codes, k_codes, kc_stride_b,
                                   kc_stride_h, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx, idx_stride_b,
                                   idx_stride_h, count, hist_out, workspace, (cudaStream_t)stream,
                                   Windows{shape->n_sink, shape->n_local}));
    return HA_OK;
}

int ha_inner_products(const uint16_t *q, const uint16_t *K, int64_t n, int64_t row_stride, float *dots, void *stream) {
    if (n < 0 || !q || (n > 0 && (!K || !dots)) || row_stride < kD || (row_stride & 7)) return HA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) & 15) || (reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(dots) & 3))
        return HA_ERR_INVALID_ARG;
    HA_CUDA(launch_inner_products(q, K, n, row_stride, dots, (cudaStream_t)stream));
    return HA_OK;
}

int ha_read_device_status(void *workspace, void *stream, uint32_t *flags) {
    if (!workspace || !flags) return HA_ERR_INVALID_ARG;
    HA_CUDA(cudaMemcpyAsync(flags, workspace, sizeof(uint32_t), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    HA_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    return HA_OK;
}

uint64_t ha_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

const char *ha_status_string(int status) {
    switch (status) {
        case HA_OK: return "ok";
        case HA_ERR_INVALID_ARG: return "invalid argument";
        case HA_ERR_UNSUPPORTED: return "unsupported configuration";
        case HA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case HA_ERR_CUDA: return "CUDA runtime error";
        case HA_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of ha_gather_attn_static (batch * n_kv_heads <= 64)";
        default: return "unknown status";
    }
}

const char *ha_version(void) { return "hashattn-b200 0.1 (sm_100a)"; }

} // extern "C"
