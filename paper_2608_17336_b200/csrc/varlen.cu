// Variable-length batches (Sec. 4.1, "grouped-query attention and variable-length batching"; App. C,
// scale shapes for variable-length batches): host-side prefix sums over the sequences, their copy
// into the workspace, and the C ABI of the three steps over a packed batch.
#include <math.h>

#include <algorithm>

#include "common.cuh"

namespace tilemix {

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool all_zero(const int64_t s[3]) { return s[0] == 0 && s[1] == 0 && s[2] == 0; }

size_t table_bytes(const VarlenTable& t) { return align_up(t.tab.size() * sizeof(int32_t), 256); }

}  // namespace

int resolve_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl, Geometry* g, VarlenTable* t) {
    if (p == nullptr || vl == nullptr || vl->cu_seqlens == nullptr) return TILEMIX_ERR_NULL;
    if (vl->n_seqs <= 0 || vl->max_seqlen < 0) return TILEMIX_ERR_SHAPE;
    if (p->batch != 1 || p->mask_batch != 1) return TILEMIX_ERR_SHAPE;
    // Flattened token-major layout [total, H, d] when no strides are given.
    tilemix_problem_t q = *p;
    if (all_zero(q.q_stride)) { q.q_stride[0] = 0; q.q_stride[1] = q.head_dim; q.q_stride[2] = int64_t(q.heads_q) * q.head_dim; }
    if (all_zero(q.k_stride)) { q.k_stride[0] = 0; q.k_stride[1] = q.head_dim; q.k_stride[2] = int64_t(q.heads_kv) * q.head_dim; }
    if (all_zero(q.v_stride)) { q.v_stride[0] = 0; q.v_stride[1] = q.head_dim; q.v_stride[2] = int64_t(q.heads_kv) * q.head_dim; }
    if (all_zero(q.o_stride)) { q.o_stride[0] = 0; q.o_stride[1] = q.head_dim; q.o_stride[2] = int64_t(q.heads_q) * q.head_dim; }
    int rc = resolve(&q, g);
    if (rc) return rc;
    // The batch stride is never used (B = 1); a token-major tensor has none worth naming, and the
    // tensor maps need a non-zero one.
    const int64_t whole_q = static_cast<int64_t>(g->L) * g->qs[2], whole_k = static_cast<int64_t>(g->L) * g->ks[2];
    g->qs[0] = whole_q; g->os[0] = static_cast<int64_t>(g->L) * g->os[2];
    g->ks[0] = whole_k; g->vs[0] = static_cast<int64_t>(g->L) * g->vs[2];

    const int n = vl->n_seqs;
    const int32_t* cu = vl->cu_seqlens;
    if (cu[0] != 0 || cu[n] != p->seqlen) return TILEMIX_ERR_SHAPE;
    t->n = n;
    t->tab.assign(4u * (static_cast<size_t>(n) + 1u), 0);
    int32_t* tok = t->tab.data();
    int32_t* tile = tok + (n + 1);
    int32_t* blkq = tile + (n + 1);
    int32_t* blkk = blkq + (n + 1);
    std::vector<int32_t> pair(static_cast<size_t>(n) + 1u, 0);
    int64_t longest = 0;
    for (int s = 0; s < n; ++s) {
        const int64_t len = static_cast<int64_t>(cu[s + 1]) - cu[s];
        if (len < 0) return TILEMIX_ERR_SHAPE;
        longest = len > longest ? len : longest;
        const int64_t rows = ceil_div(len, g->tile_m);
        tok[s] = cu[s];
        tile[s + 1] = tile[s] + static_cast<int32_t>(rows);
        pair[s + 1] = pair[s] + static_cast<int32_t>((rows + 1) / 2);
        blkq[s + 1] = blkq[s] + static_cast<int32_t>(ceil_div(len, g->blk_q));
        blkk[s + 1] = blkk[s] + static_cast<int32_t>(ceil_div(len, g->blk_k));
    }
    tok[n] = cu[n];
    if (vl->max_seqlen != 0 && vl->max_seqlen < longest) return TILEMIX_ERR_SHAPE;
    t->max_len = vl->max_seqlen != 0 ? vl->max_seqlen : static_cast<int>(longest);
    if (t->max_len <= 0) t->max_len = 1;   // only reachable with seqlen > 0, kept for safety
    t->total_tiles = tile[n];
    t->total_pairs = pair[n];
    t->total_blk_q = blkq[n];
    t->total_blk_k = blkk[n];
    // Work items of the attention kernel, the longest rows of the whole batch first (a pair p of a
    // sequence streams 2p + 2 key tiles); ties keep the sequence order.
    std::vector<std::pair<int32_t, int32_t>> items;   // (pair index, sequence)
    items.reserve(static_cast<size_t>(t->total_pairs));
    for (int s = 0; s < n; ++s)
        for (int32_t pr = pair[s + 1] - pair[s] - 1; pr >= 0; --pr) items.emplace_back(pr, s);
    std::stable_sort(items.begin(), items.end(),
                     [](const std::pair<int32_t, int32_t>& a, const std::pair<int32_t, int32_t>& b) { return a.first > b.first; });
    const size_t base = t->tab.size();
    t->tab.resize(base + 2u * items.size());
    for (size_t i = 0; i < items.size(); ++i) {
        t->tab[base + i] = items[i].second;
        t->tab[base + items.size() + i] = items[i].first;
    }
    g->T_m = t->total_tiles;
    g->mask_T_m = t->total_tiles;
    g->T_n = static_cast<int>(ceil_div(t->max_len, g->tile_n));
    g->T_mask = static_cast<int>(ceil_div(t->max_len, static_cast<int64_t>(g->G) * g->tile_n));
    g->W = static_cast<int>(ceil_div(g->T_mask, 32));
    return TILEMIX_OK;
}

int upload_varlen(const VarlenTable& t, void* workspace, cudaStream_t stream, VarlenDev* dev) {
    int32_t* base = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + kStatusAreaBytes);
    // The source is pageable host memory: the runtime has staged it by the time the call returns.
    const cudaError_t e = cudaMemcpyAsync(base, t.tab.data(), t.tab.size() * sizeof(int32_t),
                                          cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return static_cast<int>(e);
    const int n1 = t.n + 1;
    dev->tok = base; dev->tile = base + n1; dev->blkq = base + 2 * n1; dev->blkk = base + 3 * n1;
    dev->item_seq = base + 4 * n1;
    dev->item_pair = dev->item_seq + t.total_pairs;
    dev->n = t.n;
    return TILEMIX_OK;
}

}  // namespace tilemix

using namespace tilemix;

extern "C" {

int tilemix_varlen_counts(const tilemix_problem_t* p, const tilemix_varlen_t* vl, int64_t out[7]) {
    if (out == nullptr) return TILEMIX_ERR_NULL;
    Geometry g;
    VarlenTable t;
    const int rc = resolve_varlen(p, vl, &g, &t);
    if (rc) return rc;
    out[0] = g.L; out[1] = t.total_tiles; out[2] = t.total_blk_q; out[3] = t.total_blk_k;
    out[4] = g.T_mask; out[5] = g.W; out[6] = t.max_len;
    return TILEMIX_OK;
}

size_t tilemix_varlen_workspace_size(const tilemix_problem_t* p, const tilemix_varlen_t* vl) {
    Geometry g;
    VarlenTable t;
    if (resolve_varlen(p, vl, &g, &t)) return 0;
    return kStatusAreaBytes + table_bytes(t);
}

int tilemix_quantize_qk_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl, const void* q_f16,
                               const void* k_f16, int8_t* q_i8, int8_t* k_i8, float* q_scale, float* k_scale,
                               void* workspace, size_t workspace_bytes, void* stream) {
    Geometry g;
    VarlenTable t;
    int rc = resolve_varlen(p, vl, &g, &t);
    if (rc) return rc;
    const bool do_q = q_f16 || q_i8 || q_scale, do_k = k_f16 || k_i8 || k_scale;
    if ((!do_q && !do_k) || workspace == nullptr) return TILEMIX_ERR_NULL;
    if (do_q && !(q_f16 && q_i8 && q_scale)) return TILEMIX_ERR_NULL;
    if (do_k && !(k_f16 && k_i8 && k_scale)) return TILEMIX_ERR_NULL;
    if ((do_q && (!aligned16(q_f16) || !aligned16(q_i8))) || (do_k && (!aligned16(k_f16) || !aligned16(k_i8))) ||
        !aligned16(workspace))
        return TILEMIX_ERR_ALIGN;
    if (workspace_bytes < kStatusAreaBytes + table_bytes(t)) return TILEMIX_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    VarlenDev dev;
    if ((rc = upload_varlen(t, workspace, s, &dev))) return rc;
    if (do_q && t.total_blk_q > 0 &&
        (rc = launch_quantize(q_f16, g.qs, 1, g.Hq, g.L, g.d, g.blk_q, q_i8, q_scale, s, &dev, dev.blkq, t.total_blk_q)))
        return rc;
    if (do_k && t.total_blk_k > 0 &&
        (rc = launch_quantize(k_f16, g.ks, 1, g.Hk, g.L, g.d, g.blk_k, k_i8, k_scale, s, &dev, dev.blkk, t.total_blk_k)))
        return rc;
    return TILEMIX_OK;
}

int tilemix_pack_routing_mask_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl, const uint8_t* route,
                                     uint32_t pack_flags, uint32_t* mask_words, uint64_t* counts, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    Geometry g;
    VarlenTable t;
    int rc = resolve_varlen(p, vl, &g, &t);
    if (rc) return rc;
    if (route == nullptr || mask_words == nullptr || workspace == nullptr) return TILEMIX_ERR_NULL;
    if (!aligned16(workspace)) return TILEMIX_ERR_ALIGN;
    if (workspace_bytes < kStatusAreaBytes + table_bytes(t)) return TILEMIX_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    VarlenDev dev;
    if ((rc = upload_varlen(t, workspace, s, &dev))) return rc;
    return launch_pack(g, route, pack_flags, mask_words, reinterpret_cast<unsigned long long*>(counts), s, &dev);
}

int tilemix_attention_fwd_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl, const void* q_f16,
                                 const void* k_f16, const void* v_f16, const int8_t* q_i8, const int8_t* k_i8,
                                 const float* q_scale, const float* k_scale, const uint32_t* mask_words,
                                 void* out_f16, float* lse, void* workspace, size_t workspace_bytes,
                                 const tilemix_debug_t* dbg, void* stream) {
    Geometry g;
    VarlenTable t;
    int rc = resolve_varlen(p, vl, &g, &t);
    if (rc) return rc;
    if (!q_f16 || !k_f16 || !v_f16 || !out_f16 || !workspace) return TILEMIX_ERR_NULL;
    if ((g.flags & TILEMIX_QUANT_ON_THE_FLY) != 0) return TILEMIX_ERR_UNSUPPORTED;   // dense batches only
    const bool force16 = (g.flags & TILEMIX_FORCE_FP16) != 0;
    if (!force16 && !(q_i8 && k_i8 && q_scale && k_scale && mask_words)) return TILEMIX_ERR_NULL;
    if (dbg && dbg->n_tiles > 0 && !(dbg->tiles && dbg->raw && dbg->kind)) return TILEMIX_ERR_NULL;
    if (dbg && dbg->n_tiles < 0) return TILEMIX_ERR_SHAPE;
    const bool shape_ok = (g.d == 128 && g.tile_m == 128 && g.tile_n == 128) ||
                          (g.d == 64 && g.tile_m == 64 && g.tile_n == 64);
    if (!shape_ok) return TILEMIX_ERR_UNSUPPORTED;
    if (g.blk_q != g.tile_m || (g.blk_k != g.tile_n && g.blk_k * 2 != g.tile_n)) return TILEMIX_ERR_UNSUPPORTED;
    if (g.T_n > 2048) return TILEMIX_ERR_UNSUPPORTED;   // schedule table of the kernel
    if (!aligned16(q_f16) || !aligned16(k_f16) || !aligned16(v_f16) || !aligned16(out_f16) ||
        !aligned16(workspace) || (!force16 && (!aligned16(q_i8) || !aligned16(k_i8))) ||
        (dbg && dbg->n_tiles > 0 && !aligned16(dbg->raw)))
        return TILEMIX_ERR_ALIGN;
    if (workspace_bytes < kStatusAreaBytes + table_bytes(t)) return TILEMIX_ERR_WORKSPACE;
    int dev_id = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev_id);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev_id);
    if (e != cudaSuccess) return static_cast<int>(e);
    if (major != 10) return TILEMIX_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    VarlenDev dev;
    if ((rc = upload_varlen(t, workspace, s, &dev))) return rc;
    return launch_attention(g, q_f16, k_f16, v_f16, force16 ? nullptr : q_i8, force16 ? nullptr : k_i8, q_scale,
                            k_scale, mask_words, out_f16, lse, workspace, dbg, s, &dev, t.total_pairs);
}

}  // extern "C"
