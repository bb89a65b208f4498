// C ABI of libtilemix: argument validation on the host, then the kernel launchers.
#include <cuda_fp16.h>
#include <math.h>
#include <string.h>

#include <mutex>

#include "common.cuh"

namespace tilemix {

std::atomic<uint64_t> g_launch_count{0};
std::atomic<int> g_test_drop{0};
std::atomic<uint64_t> g_wait_limit_ns{kDefaultWaitLimitNs};

namespace {

bool all_zero(const int64_t s[3]) { return s[0] == 0 && s[1] == 0 && s[2] == 0; }

void dense_strides(int H, int L, int d, int64_t out[3]) {
    out[0] = static_cast<int64_t>(H) * L * d;
    out[1] = static_cast<int64_t>(L) * d;
    out[2] = d;
}

int set_strides(const int64_t in[3], int H, int L, int d, int64_t out[3]) {
    if (all_zero(in)) {
        dense_strides(H, L, d, out);
        return TILEMIX_OK;
    }
    for (int i = 0; i < 3; ++i) {
        if (in[i] < 0) return TILEMIX_ERR_SHAPE;
        out[i] = in[i];
    }
    if (out[2] < d) return TILEMIX_ERR_SHAPE;
    // 16-byte granularity of FP16 rows (vector loads and TMA global strides)
    for (int i = 0; i < 3; ++i)
        if ((out[i] * 2) % 16 != 0) return TILEMIX_ERR_ALIGN;
    return TILEMIX_OK;
}

int check_device() {
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    return major == 10 ? TILEMIX_OK : TILEMIX_ERR_UNSUPPORTED;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// What tilemix_attention_fwd and tilemix_attention_fwd_chunk check on the host before the launch (the geometry is
// resolved by the caller: the chunk entry point rewrites the key/value side of it first).
int checked_attention(const Geometry& g, const void* q_f16, const void* k_f16, const void* v_f16, const int8_t* q_i8,
                      const int8_t* k_i8, const float* q_scale, const float* k_scale, const uint32_t* mask_words,
                      void* out_f16, float* lse, void* workspace, size_t workspace_bytes, const tilemix_debug_t* dbg,
                      void* stream, const float* v_scale = nullptr) {
    if (!q_f16 || !k_f16 || !v_f16 || !out_f16 || !workspace) return TILEMIX_ERR_NULL;
    const bool force16 = (g.flags & TILEMIX_FORCE_FP16) != 0;
    const bool otf = (g.flags & TILEMIX_QUANT_ON_THE_FLY) != 0;   // INT8 operands and scales are made on chip
    if (!force16 && !otf && !(q_i8 && k_i8 && q_scale && k_scale)) return TILEMIX_ERR_NULL;
    if (!force16 && !mask_words) return TILEMIX_ERR_NULL;
    if (otf && !(g.d == 128 && g.tile_m == 128 && g.tile_n == 128)) return TILEMIX_ERR_UNSUPPORTED;
    if (dbg && dbg->n_tiles > 0 && !(dbg->tiles && dbg->raw && dbg->kind)) return TILEMIX_ERR_NULL;
    if (dbg && dbg->n_tiles < 0) return TILEMIX_ERR_SHAPE;
    const bool shape_ok = (g.d == 128 && g.tile_m == 128 && g.tile_n == 128) ||
                          (g.d == 64 && g.tile_m == 64 && g.tile_n == 64);
    if (!shape_ok) return TILEMIX_ERR_UNSUPPORTED;
    // quantisation blocks: Q per query tile; K per key tile or per half key tile (App. C: BLK_K = BLOCK_N / 2)
    if (g.blk_q != g.tile_m || (g.blk_k != g.tile_n && g.blk_k * 2 != g.tile_n)) return TILEMIX_ERR_UNSUPPORTED;
    if (otf && g.blk_k != g.tile_n) return TILEMIX_ERR_UNSUPPORTED;   // the on-chip quantiser works per key tile
    if (g.T_n > 2048) return TILEMIX_ERR_UNSUPPORTED;   // schedule table of the kernel
    if (!aligned16(q_f16) || !aligned16(k_f16) || !aligned16(v_f16) || !aligned16(out_f16) ||
        !aligned16(workspace) || (!force16 && (!aligned16(q_i8) || !aligned16(k_i8))) ||
        (dbg && dbg->n_tiles > 0 && !aligned16(dbg->raw)))
        return TILEMIX_ERR_ALIGN;
    if (workspace_bytes < kStatusAreaBytes) return TILEMIX_ERR_WORKSPACE;
    const int rc = check_device();
    if (rc) return rc;
    return launch_attention(g, q_f16, k_f16, v_f16, force16 ? nullptr : q_i8, force16 ? nullptr : k_i8, q_scale,
                            k_scale, mask_words, out_f16, lse, workspace, dbg, static_cast<cudaStream_t>(stream),
                            nullptr, 0, v_scale);
}

// INT8 value cache -> its exact FP16 image (|x| <= 127 is exact in binary16), 16 values per thread.
__global__ void v8_to_f16_kernel(const int8_t* __restrict__ v8, __half* __restrict__ v16, int64_t n16) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n16) return;
    const uint4 in = reinterpret_cast<const uint4*>(v8)[i];
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    uint32_t h[8];
#pragma unroll
    for (int y = 0; y < 4; ++y) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int lo = static_cast<int8_t>(w[y] >> (16 * e)), hi = static_cast<int8_t>(w[y] >> (16 * e + 8));
            const __half2 v = __floats2half2_rn(static_cast<float>(lo), static_cast<float>(hi));
            h[2 * y + e] = *reinterpret_cast<const uint32_t*>(&v);
        }
    }
    uint4* out = reinterpret_cast<uint4*>(v16) + 2 * i;
    out[0] = make_uint4(h[0], h[1], h[2], h[3]);
    out[1] = make_uint4(h[4], h[5], h[6], h[7]);
}

// Geometry of a chunk of the last p->seqlen tokens of a kv_len-token context (K and V are kv_len tokens long).
int resolve_chunk(const tilemix_problem_t* p, int32_t kv_len, Geometry* g) {
    if (p == nullptr) return TILEMIX_ERR_NULL;
    if (kv_len < p->seqlen || p->tile_m <= 0 || p->tile_m != p->tile_n || (kv_len - p->seqlen) % p->tile_m != 0)
        return TILEMIX_ERR_SHAPE;
    // K and V are kv_len tokens long: dense strides are theirs, not the chunk's
    tilemix_problem_t q = *p;
    if (all_zero(q.k_stride)) dense_strides(q.heads_kv, kv_len, q.head_dim, q.k_stride);
    if (all_zero(q.v_stride)) dense_strides(q.heads_kv, kv_len, q.head_dim, q.v_stride);
    const int rc = resolve(&q, g);
    if (rc) return rc;
    g->Lk = kv_len;
    g->kv_off = (kv_len - g->L) / g->tile_m;
    g->T_n = static_cast<int>(ceil_div(kv_len, g->tile_n));
    g->mask_T_m = g->T_n;                      // the mask words of the whole context
    g->ks_blocks = static_cast<int>(ceil_div(kv_len, g->blk_k));
    g->T_mask = static_cast<int>(ceil_div(kv_len, static_cast<int64_t>(g->G) * g->tile_n));
    g->W = static_cast<int>(ceil_div(g->T_mask, 32));
    return TILEMIX_OK;
}

}  // namespace

int resolve(const tilemix_problem_t* p, Geometry* g) {
    if (p == nullptr) return TILEMIX_ERR_NULL;
    if (p->batch <= 0 || p->heads_q <= 0 || p->heads_kv <= 0 || p->seqlen <= 0 || p->head_dim <= 0 ||
        p->tile_m <= 0 || p->tile_n <= 0 || p->group <= 0)
        return TILEMIX_ERR_SHAPE;
    if (p->heads_q % p->heads_kv != 0) return TILEMIX_ERR_SHAPE;
    if (p->head_dim % 8 != 0) return TILEMIX_ERR_SHAPE;
    if (p->mask_batch != 1 && p->mask_batch != p->batch) return TILEMIX_ERR_SHAPE;
    if (p->quant_blk_q < 0 || p->quant_blk_k < 0) return TILEMIX_ERR_SHAPE;
    g->B = p->batch; g->Hq = p->heads_q; g->Hk = p->heads_kv; g->L = p->seqlen; g->d = p->head_dim;
    g->tile_m = p->tile_m; g->tile_n = p->tile_n; g->G = p->group;
    g->blk_q = p->quant_blk_q ? p->quant_blk_q : p->tile_m;
    g->blk_k = p->quant_blk_k ? p->quant_blk_k : p->tile_n;
    g->nb = p->mask_batch;
    g->T_m = static_cast<int>(ceil_div(g->L, g->tile_m));
    g->T_n = static_cast<int>(ceil_div(g->L, g->tile_n));
    g->T_mask = static_cast<int>(ceil_div(g->L, static_cast<int64_t>(g->G) * g->tile_n));
    g->W = static_cast<int>(ceil_div(g->T_mask, 32));
    g->Lk = g->L; g->kv_off = 0; g->mask_T_m = g->T_m; g->ks_blocks = static_cast<int>(ceil_div(g->L, g->blk_k));
    g->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf(static_cast<float>(g->d));
    g->flags = p->flags;
    int rc;
    if ((rc = set_strides(p->q_stride, g->Hq, g->L, g->d, g->qs))) return rc;
    if ((rc = set_strides(p->k_stride, g->Hk, g->L, g->d, g->ks))) return rc;
    if ((rc = set_strides(p->v_stride, g->Hk, g->L, g->d, g->vs))) return rc;
    if ((rc = set_strides(p->o_stride, g->Hq, g->L, g->d, g->os))) return rc;
    return TILEMIX_OK;
}

}  // namespace tilemix

using namespace tilemix;

extern "C" {

int tilemix_quantize_qk(const tilemix_problem_t* p, const void* q_f16, const void* k_f16, int8_t* q_i8,
                        int8_t* k_i8, float* q_scale, float* k_scale, void* stream) {
    Geometry g;
    int rc = resolve(p, &g);
    if (rc) return rc;
    const bool do_q = q_f16 || q_i8 || q_scale, do_k = k_f16 || k_i8 || k_scale;
    if (!do_q && !do_k) return TILEMIX_ERR_NULL;
    if (do_q && !(q_f16 && q_i8 && q_scale)) return TILEMIX_ERR_NULL;
    if (do_k && !(k_f16 && k_i8 && k_scale)) return TILEMIX_ERR_NULL;
    if ((do_q && (!aligned16(q_f16) || !aligned16(q_i8))) || (do_k && (!aligned16(k_f16) || !aligned16(k_i8))))
        return TILEMIX_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (do_q && do_k)
        return launch_quantize_pair(q_f16, g.qs, g.Hq, g.blk_q, q_i8, q_scale, k_f16, g.ks, g.Hk, g.blk_k, k_i8, k_scale,
                                    g.B, g.L, g.d, s);
    if (do_q && (rc = launch_quantize(q_f16, g.qs, g.B, g.Hq, g.L, g.d, g.blk_q, q_i8, q_scale, s))) return rc;
    if (do_k && (rc = launch_quantize(k_f16, g.ks, g.B, g.Hk, g.L, g.d, g.blk_k, k_i8, k_scale, s))) return rc;
    return TILEMIX_OK;
}

int tilemix_pack_routing_mask(const tilemix_problem_t* p, const uint8_t* route, uint32_t pack_flags,
                              uint32_t* mask_words, uint64_t* counts, void* stream) {
    Geometry g;
    int rc = resolve(p, &g);
    if (rc) return rc;
    if (route == nullptr || mask_words == nullptr) return TILEMIX_ERR_NULL;
    return launch_pack(g, route, pack_flags, mask_words, reinterpret_cast<unsigned long long*>(counts),
                       static_cast<cudaStream_t>(stream));
}

int tilemix_attention_fwd(const tilemix_problem_t* p, const void* q_f16, const void* k_f16, const void* v_f16,
                          const int8_t* q_i8, const int8_t* k_i8, const float* q_scale, const float* k_scale,
                          const uint32_t* mask_words, void* out_f16, float* lse, void* workspace,
                          size_t workspace_bytes, const tilemix_debug_t* dbg, void* stream) {
    Geometry g;
    int rc = resolve(p, &g);
    if (rc) return rc;
    return checked_attention(g, q_f16, k_f16, v_f16, q_i8, k_i8, q_scale, k_scale, mask_words, out_f16, lse, workspace,
                             workspace_bytes, dbg, stream);
}

int tilemix_attention_fwd_chunk(const tilemix_problem_t* p, int32_t kv_len, const void* q_f16, const void* k_f16,
                                const void* v_f16, const int8_t* q_i8, const int8_t* k_i8, const float* q_scale,
                                const float* k_scale, const uint32_t* mask_words, void* out_f16, float* lse,
                                void* workspace, size_t workspace_bytes, const tilemix_debug_t* dbg, void* stream) {
    Geometry g;
    const int rc = resolve_chunk(p, kv_len, &g);
    if (rc) return rc;
    return checked_attention(g, q_f16, k_f16, v_f16, q_i8, k_i8, q_scale, k_scale, mask_words, out_f16, lse, workspace,
                             workspace_bytes, dbg, stream);
}

size_t tilemix_chunk_v8_workspace_size(const tilemix_problem_t* p, int32_t kv_len) {
    Geometry g;
    if (resolve_chunk(p, kv_len, &g)) return 0;
    return kStatusAreaBytes + static_cast<size_t>(g.B) * g.Hk * g.Lk * g.d * sizeof(__half);
}

int tilemix_attention_fwd_chunk_v8(const tilemix_problem_t* p, int32_t kv_len, const void* q_f16, const void* k_f16,
                                   const int8_t* v_i8, const float* v_scale, const int8_t* q_i8, const int8_t* k_i8,
                                   const float* q_scale, const float* k_scale, const uint32_t* mask_words,
                                   void* out_f16, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (p == nullptr) return TILEMIX_ERR_NULL;
    tilemix_problem_t q = *p;
    for (int i = 0; i < 3; ++i) q.v_stride[i] = 0;     // the INT8 value cache is dense; so is its FP16 image
    Geometry g;
    int rc = resolve_chunk(&q, kv_len, &g);
    if (rc) return rc;
    if (!v_i8 || !v_scale || !workspace) return TILEMIX_ERR_NULL;
    if (g.flags & TILEMIX_QUANT_ON_THE_FLY) return TILEMIX_ERR_UNSUPPORTED;
    if (!aligned16(v_i8) || !aligned16(workspace)) return TILEMIX_ERR_ALIGN;
    const size_t n = static_cast<size_t>(g.B) * g.Hk * g.Lk * g.d;
    if (workspace_bytes < kStatusAreaBytes + n * sizeof(__half)) return TILEMIX_ERR_WORKSPACE;
    if ((rc = check_device())) return rc;
    __half* v16 = reinterpret_cast<__half*>(static_cast<uint8_t*>(workspace) + kStatusAreaBytes);
    const int64_t n16 = static_cast<int64_t>(n / 16);  // head_dim is 64 or 128: whole 16-byte pieces
    if (n16 > 0) {
        v8_to_f16_kernel<<<static_cast<unsigned>((n16 + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(v_i8, v16, n16);
        g_launch_count.fetch_add(1);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return static_cast<int>(e);
    }
    return checked_attention(g, q_f16, k_f16, v16, q_i8, k_i8, q_scale, k_scale, mask_words, out_f16, lse, workspace,
                             kStatusAreaBytes, nullptr, stream, v_scale);
}

int tilemix_mask_words_per_row(int seqlen, int tile_n, int group) {
    if (seqlen <= 0 || tile_n <= 0 || group <= 0) return TILEMIX_ERR_SHAPE;
    const int64_t t_mask = ceil_div(seqlen, static_cast<int64_t>(tile_n) * group);
    return static_cast<int>(ceil_div(t_mask, 32));
}

size_t tilemix_workspace_size(const tilemix_problem_t* p) {
    Geometry g;
    if (resolve(p, &g)) return 0;
    return kStatusAreaBytes;   // status record (16 bytes) at the start
}

size_t tilemix_scratch_bytes(const tilemix_problem_t* p) {
    Geometry g;
    if (resolve(p, &g)) return 0;
    const size_t int8 = static_cast<size_t>(g.B) * g.L * g.d * (static_cast<size_t>(g.Hq) + g.Hk);
    const size_t scales = 4u * static_cast<size_t>(g.B) *
                          (static_cast<size_t>(g.Hq) * ceil_div(g.L, g.blk_q) + static_cast<size_t>(g.Hk) * ceil_div(g.L, g.blk_k));
    const size_t words = 4u * static_cast<size_t>(g.nb) * g.Hk * g.T_m * g.W;
    return int8 + scales + words;
}

namespace {
// Layout of the arena used by tilemix_prefill_host (every region 256-byte aligned).
struct Arena {
    size_t q, k, v, o, q8, k8, qs, ks, route, words, work, total;
};
Arena arena_layout(const Geometry& g) {
    Arena a;
    size_t off = 0;
    auto put = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
    const size_t nq = static_cast<size_t>(g.B) * g.Hq * g.L * g.d, nk = static_cast<size_t>(g.B) * g.Hk * g.L * g.d;
    a.q = put(nq * 2); a.k = put(nk * 2); a.v = put(nk * 2); a.o = put(nq * 2);
    a.q8 = put(nq); a.k8 = put(nk);
    a.qs = put(4u * static_cast<size_t>(g.B) * g.Hq * ceil_div(g.L, g.blk_q));
    a.ks = put(4u * static_cast<size_t>(g.B) * g.Hk * ceil_div(g.L, g.blk_k));
    a.route = put(static_cast<size_t>(g.nb) * g.Hk * g.T_m * g.T_mask);
    a.words = put(4u * static_cast<size_t>(g.nb) * g.Hk * g.T_m * g.W);
    a.work = put(4096);
    a.total = off;
    return a;
}
}  // namespace

size_t tilemix_arena_size(const tilemix_problem_t* p) {
    Geometry g;
    if (resolve(p, &g)) return 0;
    return arena_layout(g).total;
}

namespace {

// Helper streams and events of tilemix_prefill_host, created on first use per device and kept until
// the process exits (stream/event creation is not a device-memory allocation and does not synchronise).
constexpr int kMaxChunks = 8;
struct HostPipe {
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, landed[kMaxChunks] = {}, done[kMaxChunks] = {}, drained = nullptr;
};
HostPipe g_pipe[64];
std::mutex g_pipe_mutex[64];   // one call at a time per device enqueues on the helper streams

// Called with g_pipe_mutex[dev] held.
int host_pipe(int dev, HostPipe** out) {
    HostPipe& hp = g_pipe[dev];
    int rc = TILEMIX_OK;
    if (!hp.ready) {
        auto ev = [&](cudaEvent_t* x) { if (rc == 0) rc = static_cast<int>(cudaEventCreateWithFlags(x, cudaEventDisableTiming)); };
        if (rc == 0) rc = static_cast<int>(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
        if (rc == 0) rc = static_cast<int>(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
        ev(&hp.start); ev(&hp.drained);
        for (int i = 0; i < kMaxChunks; ++i) { ev(&hp.landed[i]); ev(&hp.done[i]); }
        hp.ready = rc == 0;
    }
    *out = &hp;
    return rc;
}

}  // namespace

int tilemix_prefill_host(const tilemix_problem_t* p, const void* q_host, const void* k_host, const void* v_host,
                         const uint8_t* route_host, uint32_t pack_flags, void* out_host, void* arena,
                         size_t arena_bytes, void* stream) {
    Geometry g;
    int rc = resolve(p, &g);
    if (rc) return rc;
    if (!q_host || !k_host || !v_host || !route_host || !out_host || !arena) return TILEMIX_ERR_NULL;
    if (!all_zero(p->q_stride) || !all_zero(p->k_stride) || !all_zero(p->v_stride) || !all_zero(p->o_stride))
        return TILEMIX_ERR_UNSUPPORTED;   // host buffers are dense
    if (reinterpret_cast<uintptr_t>(arena) % 256 != 0) return TILEMIX_ERR_ALIGN;
    const Arena a = arena_layout(g);
    if (arena_bytes < a.total) return TILEMIX_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* base = static_cast<uint8_t*>(arena);
    // The helper streams and events belong to the device, so the whole enqueue below is one critical section per
    // device: calls from several host threads (on any streams) are enqueued one after the other, never interleaved.
    int dev = 0;
    if (cudaError_t de = cudaGetDevice(&dev); de != cudaSuccess) return static_cast<int>(de);
    if (dev < 0 || dev >= 64) return TILEMIX_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> enqueue_lock(g_pipe_mutex[dev]);
    HostPipe* hp = nullptr;
    if ((rc = host_pipe(dev, &hp))) return rc;

    // The batch (or, for one sequence, its KV heads) is cut into chunks that flow through three
    // engines at once: host->device copies on a helper stream, the three kernels on the caller's
    // stream, device->host copies on a second helper stream.  Everything is ordered behind what the
    // caller's stream held on entry, and the caller's stream ends up behind the last copy.
    const bool by_batch = g.B > 1;
    const int units = by_batch ? g.B : g.Hk;
    const int per_chunk = static_cast<int>(ceil_div(units, kMaxChunks));
    const int n_chunks = static_cast<int>(ceil_div(units, per_chunk));
    const int rep = g.Hq / g.Hk;
    const size_t head_elems = static_cast<size_t>(g.L) * g.d;
    cudaError_t e;
    if ((e = cudaEventRecord(hp->start, s)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(hp->in, hp->start, 0)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(hp->out, hp->start, 0)) != cudaSuccess) return e;
    // routing map: small, copied and packed once for the whole problem
    if ((e = cudaMemcpyAsync(base + a.route, route_host, static_cast<size_t>(g.nb) * g.Hk * g.T_m * g.T_mask,
                             cudaMemcpyHostToDevice, s)) != cudaSuccess)
        return e;
    if ((rc = tilemix_pack_routing_mask(p, base + a.route, pack_flags, reinterpret_cast<uint32_t*>(base + a.words),
                                        nullptr, stream)))
        return rc;
    for (int c = 0; c < n_chunks; ++c) {
        const int u0 = c * per_chunk, nu = (u0 + per_chunk <= units ? per_chunk : units - u0);
        // element offsets of the chunk inside the dense [B, H, L, d] tensors, and its byte counts
        const size_t q_off = by_batch ? static_cast<size_t>(u0) * g.Hq * head_elems : static_cast<size_t>(u0) * rep * head_elems;
        const size_t k_off = by_batch ? static_cast<size_t>(u0) * g.Hk * head_elems : static_cast<size_t>(u0) * head_elems;
        const size_t q_n = by_batch ? static_cast<size_t>(nu) * g.Hq * head_elems : static_cast<size_t>(nu) * rep * head_elems;
        const size_t k_n = by_batch ? static_cast<size_t>(nu) * g.Hk * head_elems : static_cast<size_t>(nu) * head_elems;
        const uint8_t* qh = static_cast<const uint8_t*>(q_host) + q_off * 2;
        const uint8_t* kh = static_cast<const uint8_t*>(k_host) + k_off * 2;
        const uint8_t* vh = static_cast<const uint8_t*>(v_host) + k_off * 2;
        if ((e = cudaMemcpyAsync(base + a.q + q_off * 2, qh, q_n * 2, cudaMemcpyHostToDevice, hp->in)) != cudaSuccess) return e;
        if ((e = cudaMemcpyAsync(base + a.k + k_off * 2, kh, k_n * 2, cudaMemcpyHostToDevice, hp->in)) != cudaSuccess) return e;
        if ((e = cudaMemcpyAsync(base + a.v + k_off * 2, vh, k_n * 2, cudaMemcpyHostToDevice, hp->in)) != cudaSuccess) return e;
        if ((e = cudaEventRecord(hp->landed[c], hp->in)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(s, hp->landed[c], 0)) != cudaSuccess) return e;
        // the chunk as a problem of its own: a batch range (dense) or a head range (strides of the whole)
        tilemix_problem_t sub = *p;
        size_t words_off = 0, qs_off = 0, ks_off = 0;
        if (by_batch) {
            sub.batch = nu;
            sub.mask_batch = g.nb == 1 ? 1 : nu;
            words_off = g.nb == 1 ? 0 : static_cast<size_t>(u0) * g.Hk * g.T_m * g.W;
            qs_off = static_cast<size_t>(u0) * g.Hq * ceil_div(g.L, g.blk_q);
            ks_off = static_cast<size_t>(u0) * g.Hk * ceil_div(g.L, g.blk_k);
        } else {
            sub.heads_kv = nu;
            sub.heads_q = nu * rep;
            for (int t = 0; t < 3; ++t) {
                sub.q_stride[t] = g.qs[t]; sub.k_stride[t] = g.ks[t]; sub.v_stride[t] = g.vs[t]; sub.o_stride[t] = g.os[t];
            }
            words_off = static_cast<size_t>(u0) * g.T_m * g.W;
            qs_off = static_cast<size_t>(u0) * rep * ceil_div(g.L, g.blk_q);
            ks_off = static_cast<size_t>(u0) * ceil_div(g.L, g.blk_k);
        }
        int8_t* q8 = reinterpret_cast<int8_t*>(base + a.q8) + q_off;
        int8_t* k8 = reinterpret_cast<int8_t*>(base + a.k8) + k_off;
        float* qs = reinterpret_cast<float*>(base + a.qs) + qs_off;
        float* ks = reinterpret_cast<float*>(base + a.ks) + ks_off;
        // (the on-the-fly operand mode has no quantiser pass: the attention kernel ignores q8 .. ks)
        if (!(g.flags & TILEMIX_QUANT_ON_THE_FLY) &&
            (rc = tilemix_quantize_qk(&sub, base + a.q + q_off * 2, base + a.k + k_off * 2, q8, k8, qs, ks, stream)))
            return rc;
        if ((rc = tilemix_attention_fwd(&sub, base + a.q + q_off * 2, base + a.k + k_off * 2, base + a.v + k_off * 2, q8, k8,
                                        qs, ks, reinterpret_cast<uint32_t*>(base + a.words) + words_off,
                                        base + a.o + q_off * 2, nullptr, base + a.work, 4096, nullptr, stream)))
            return rc;
        if ((e = cudaEventRecord(hp->done[c], s)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(hp->out, hp->done[c], 0)) != cudaSuccess) return e;
        if ((e = cudaMemcpyAsync(static_cast<uint8_t*>(out_host) + q_off * 2, base + a.o + q_off * 2, q_n * 2,
                                 cudaMemcpyDeviceToHost, hp->out)) != cudaSuccess)
            return e;
    }
    if ((e = cudaEventRecord(hp->drained, hp->out)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(s, hp->drained, 0)) != cudaSuccess) return e;
    return TILEMIX_OK;
}

int tilemix_read_status(const void* workspace, int32_t out[4], void* stream) {
    if (!workspace || !out) return TILEMIX_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(out, workspace, 16, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return static_cast<int>(e);
    return out[0];
}

const char* tilemix_status_string(int code) {
    switch (code) {
        case TILEMIX_OK: return "ok";
        case TILEMIX_ERR_NULL: return "a required pointer is NULL";
        case TILEMIX_ERR_SHAPE: return "invalid shape";
        case TILEMIX_ERR_UNSUPPORTED: return "unsupported tile/head_dim combination or device";
        case TILEMIX_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
        case TILEMIX_ERR_WORKSPACE: return "workspace too small";
        case TILEMIX_ERR_DEVICE_TIMEOUT: return "a bounded wait inside the kernel ran out";
        default: return code > 0 ? cudaGetErrorString(static_cast<cudaError_t>(code)) : "unknown";
    }
}

uint64_t tilemix_launch_count(void) { return g_launch_count.load(); }

int tilemix_test_drop_copy(int which, uint64_t wait_limit_ns) {
    if (which < 0 || which > 3) return TILEMIX_ERR_SHAPE;
    g_test_drop.store(which);
    g_wait_limit_ns.store(which == 0 || wait_limit_ns == 0 ? kDefaultWaitLimitNs : wait_limit_ns);
    return TILEMIX_OK;
}

}  // extern "C"
