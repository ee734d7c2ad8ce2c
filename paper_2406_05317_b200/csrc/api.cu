// C ABI of the LoCoCo chunk-step library: argument validation, workspace layout and
// the host side of Algorithm 2's chunk loop. All arithmetic runs in the kernels.
#include <cmath>
#include <cstring>
#include <new>

#include "common.cuh"
#include "handle.h"

using namespace lococo;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A usable tensor view: non-null, 16-byte aligned base and strides.
bool view_ok(const lococo_tensor& t, size_t elt) {
    if (!t.ptr || !aligned16(t.ptr)) return false;
    if ((t.stride_batch * (int64_t)elt) % 16 || (t.stride_head * (int64_t)elt) % 16 || (t.stride_token * (int64_t)elt) % 16)
        return false;
    return t.stride_token > 0;
}

View dev(const lococo_tensor& t) { return View{static_cast<char*>(t.ptr), t.stride_batch, t.stride_head, t.stride_token}; }

View offset_tokens(const lococo_tensor& t, int64_t tokens, size_t elt) {
    View v = dev(t);
    v.ptr += tokens * t.stride_token * (int64_t)elt;
    return v;
}

lococo_tensor contiguous(void* ptr, int heads, int tokens, int d) {
    return lococo_tensor{ptr, (int64_t)heads * tokens * d, (int64_t)tokens * d, (int64_t)d};
}

void layout_workspace(lococo_handle* h) {
    const lococo_config& c = h->cfg;
    const size_t sets = c.weights_per_head ? c.heads : 1;
    const size_t Smax = (size_t)c.M + c.max_chunk;
    size_t off = 0;
    h->off_status = off;  off += 256;
    h->off_gpack = off;   off = align_up(off + sets * c.k * c.M * c.c_in * h->elt, 256);
    h->off_bias = off;    off = align_up(off + sets * c.M * sizeof(float), 256);
    h->off_s = off;       off = align_up(off + (size_t)h->units * c.M * sizeof(float), 256);
    h->off_UK = off;      off = align_up(off + (size_t)h->units * c.M * c.head_dim * sizeof(float), 256);
    h->off_UV = off;      off = align_up(off + (size_t)h->units * c.M * c.head_dim * sizeof(float), 256);
    h->off_R = off;       off = align_up(off + (size_t)h->units * c.M * Smax * sizeof(float), 256);
    tensor_layout_workspace(h, &off);
    h->ws_need = off;
}

lococo_status ready(const lococo_handle* h) {
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    if (!h->ws || !h->weights_set) return LOCOCO_ERR_WORKSPACE;
    return LOCOCO_OK;
}

// The cached loop graph holds workspace pointers and the bias choice: drop it when they change.
void drop_loop_graph(lococo_handle* h) {
    if (h->loop_graph.exec) cudaGraphExecDestroy(h->loop_graph.exec);
    h->loop_graph.exec = nullptr;
    h->loop_graph.key_len = 0;
    h->loop_graph.seen = 0;
}

lococo_status count(lococo_handle* h, int launched) {
    if (launched < 0) return LOCOCO_ERR_CUDA;
    h->launches += launched;
    return LOCOCO_OK;
}

CompressParams make_compress_params(lococo_handle* h, View kc, View vc, int c, View kn, View vn, int b, View ko, View vo,
                                    float* W_out) {
    const lococo_config& cfg = h->cfg;
    CompressParams p{};
    p.xk = CatView{kc, kn, c, b};
    p.xv = CatView{vc, vn, c, b};
    p.k_out = ko;
    p.v_out = vo;
    p.heads = cfg.heads; p.units = h->units; p.d = cfg.head_dim; p.M = cfg.M; p.k = cfg.k; p.c_in = cfg.c_in;
    p.S = c + b;
    p.weights_per_head = cfg.weights_per_head;
    p.g_packed = h->ws + h->off_gpack;
    p.bias = h->has_bias ? reinterpret_cast<const float*>(h->ws + h->off_bias) : nullptr;
    p.eps = cfg.norm_eps;
    p.prot = h->prot;
    p.R = reinterpret_cast<float*>(h->ws + h->off_R);
    p.s = reinterpret_cast<float*>(h->ws + h->off_s);
    p.UK = reinterpret_cast<float*>(h->ws + h->off_UK);
    p.UV = reinterpret_cast<float*>(h->ws + h->off_UV);
    p.W_out = W_out;
    p.prof = h->prof.on ? &h->prof : nullptr;
    return p;
}

AttnParams make_attn_params(lococo_handle* h, View q, View kc, View vc, int c, View kn, View vn, int b, View o, float* lse,
                            int64_t lse_stride) {
    const lococo_config& cfg = h->cfg;
    AttnParams p{};
    p.q = q; p.o = o;
    p.xk = CatView{kc, kn, c, b};
    p.xv = CatView{vc, vn, c, b};
    p.heads = cfg.heads; p.units = h->units; p.d = cfg.head_dim; p.b = b; p.c = c;
    p.scale = h->scale;
    p.lse = lse; p.lse_stride = lse_stride;
    p.prof = h->prof.on ? &h->prof : nullptr;
    return p;
}

lococo_status compress_impl(lococo_handle* h, View kc, View vc, int c, View kn, View vn, int b, View ko, View vo,
                            float* W_out, cudaStream_t st) {
    const lococo_config& cfg = h->cfg;
    if (c + b <= cfg.M) {
        // fill branch of Algorithm 2; carry the old rows over when the output is another buffer
        if (ko.ptr != kc.ptr || vo.ptr != vc.ptr) {
            if (c > 0) {
                FillParams f{kc, vc, ko, vo, cfg.heads, h->units, cfg.head_dim, 0, c};
                lococo_status s = count(h, simt_fill(cfg.dtype, f, st));
                if (s) return s;
            }
        }
        FillParams f{kn, vn, ko, vo, cfg.heads, h->units, cfg.head_dim, c, b};
        return count(h, simt_fill(cfg.dtype, f, st));
    }
    const CompressParams p = make_compress_params(h, kc, vc, c, kn, vn, b, ko, vo, W_out);
    if (h->use_tensor && tensor_compress_supported(h, p)) return count(h, tensor_compress(h, p, st));
    return count(h, simt_compress(cfg.dtype, p, st));
}

lococo_status attention_impl(lococo_handle* h, View q, View kc, View vc, int c, View kn, View vn, int b, View o,
                             float* lse, int64_t lse_stride, cudaStream_t st) {
    const AttnParams p = make_attn_params(h, q, kc, vc, c, kn, vn, b, o, lse, lse_stride);
    if (h->use_tensor && tensor_attention_supported(h, p)) return count(h, tensor_attention(h, p, st));
    return count(h, simt_attention(h->cfg.dtype, p, st));
}

// One step of Algorithm 2's loop: Step 3 with the old cache (kc, vc), then the update into (ko, vo), which
// may be the old cache itself. On the tensor-core path both run as one launch (they are independent of
// each other; with a separate output cache the compress CTAs can write it directly).
lococo_status step_impl(lococo_handle* h, View q, View kc, View vc, int c, View kn, View vn, int b, View o, float* lse,
                        int64_t lse_stride, View ko, View vo, cudaStream_t st) {
    if (h->use_tensor && c + b > h->cfg.M) {
        const AttnParams a = make_attn_params(h, q, kc, vc, c, kn, vn, b, o, lse, lse_stride);
        const CompressParams p = make_compress_params(h, kc, vc, c, kn, vn, b, ko, vo, nullptr);
        if (tensor_attention_supported(h, a) && tensor_compress_supported(h, p)) return count(h, tensor_chunk_step(h, a, p, st));
    }
    lococo_status s = attention_impl(h, q, kc, vc, c, kn, vn, b, o, lse, lse_stride, st);
    if (s) return s;
    return compress_impl(h, kc, vc, c, kn, vn, b, ko, vo, nullptr, st);
}

bool chunk_args_ok(const lococo_handle* h, int c, int b) {
    return c >= 0 && c <= h->cfg.M && b >= 1 && b <= h->cfg.max_chunk;
}

}  // namespace

namespace lococo {

void Profiler::begin(int kind, cudaStream_t st) {
    if (used == recs.size()) {
        Rec r{nullptr, nullptr, kind};
        if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) { on = false; return; }
        recs.push_back(r);
    }
    recs[used].kind = kind;
    cudaEventRecord(recs[used].a, st);
}
void Profiler::end(cudaStream_t st) {
    if (used < recs.size()) cudaEventRecord(recs[used++].b, st);
}
void Profiler::release() {
    for (Rec& r : recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    recs.clear();
    used = 0;
}
void prof_begin(void* p, int kind, cudaStream_t st) {
    if (p && static_cast<Profiler*>(p)->on) static_cast<Profiler*>(p)->begin(kind, st);
}
void prof_end(void* p, cudaStream_t st) {
    if (p && static_cast<Profiler*>(p)->on) static_cast<Profiler*>(p)->end(st);
}

}  // namespace lococo

extern "C" {

lococo_status lococo_profile_enable(lococo_handle* h, int32_t on) {
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    h->prof.on = on != 0;
    h->prof.used = 0;
    return LOCOCO_OK;
}

lococo_status lococo_profile_read(lococo_handle* h, int32_t kind, double* total_ms, int64_t* launches) {
    if (!h || !total_ms || !launches || kind < 0 || kind >= PROF_KINDS) return LOCOCO_ERR_INVALID_ARG;
    double ms = 0.0;
    int64_t n = 0;
    for (size_t i = 0; i < h->prof.used; ++i) {
        const Profiler::Rec& r = h->prof.recs[i];
        if (r.kind != kind) continue;
        if (cudaEventSynchronize(r.b) != cudaSuccess) return LOCOCO_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) return LOCOCO_ERR_CUDA;
        ms += t;
        ++n;
    }
    *total_ms = ms;
    *launches = n;
    return LOCOCO_OK;
}


const char* lococo_status_string(lococo_status s) {
    switch (s) {
        case LOCOCO_OK: return "ok";
        case LOCOCO_ERR_INVALID_ARG: return "invalid argument";
        case LOCOCO_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case LOCOCO_ERR_WORKSPACE: return "workspace missing or too small, or weights not set";
        case LOCOCO_ERR_CUDA: return "CUDA runtime error";
        case LOCOCO_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

lococo_status lococo_create(const lococo_config* c, lococo_handle** out) {
    if (!c || !out) return LOCOCO_ERR_INVALID_ARG;
    *out = nullptr;
    if (c->batch < 1 || c->heads < 1 || c->M < 1 || c->max_chunk < 1) return LOCOCO_ERR_INVALID_ARG;
    if (c->k < 1 || c->k % 2 == 0) return LOCOCO_ERR_INVALID_ARG;
    if (c->dtype != LOCOCO_F32 && c->dtype != LOCOCO_BF16) return LOCOCO_ERR_INVALID_ARG;
    if (c->c_in != c->head_dim && c->c_in != 2 * c->head_dim) return LOCOCO_ERR_INVALID_ARG;
    if (c->weights_per_head != 0 && c->weights_per_head != 1) return LOCOCO_ERR_INVALID_ARG;
    if (c->path < LOCOCO_PATH_AUTO || c->path > LOCOCO_PATH_TENSOR_PERSISTENT) return LOCOCO_ERR_INVALID_ARG;
    if (!(c->norm_eps >= 0.f) || !(c->softmax_scale >= 0.f)) return LOCOCO_ERR_INVALID_ARG;
    if (c->head_dim != 64 && c->head_dim != 128) return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    if (c->k > 63) return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    if ((int64_t)c->batch * c->heads > 65535) return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    if ((int64_t)c->M + c->max_chunk > (1 << 24)) return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    lococo_handle* h = new (std::nothrow) lococo_handle();
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    h->cfg = *c;
    h->units = c->batch * c->heads;
    h->elt = c->dtype == LOCOCO_F32 ? 4 : 2;
    h->scale = c->softmax_scale > 0.f ? c->softmax_scale : 1.0f / std::sqrt((float)c->head_dim);
    const bool tensor_ok = tensor_config_supported(c);
    if (c->path >= LOCOCO_PATH_TENSOR && !tensor_ok) {
        delete h;
        return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    }
    h->use_tensor = tensor_ok && c->path != LOCOCO_PATH_SIMT;
    h->persistent_loop = c->path == LOCOCO_PATH_TENSOR_PERSISTENT;
    layout_workspace(h);
    *out = h;
    return LOCOCO_OK;
}

lococo_status lococo_destroy(lococo_handle* h) {
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    h->prof.release();
    if (h->loop_graph.exec) cudaGraphExecDestroy(h->loop_graph.exec);
    tensor_sequence_release(h);
    for (int i = 0; i < h->host_ev_n; ++i) cudaEventDestroy(h->host_ev[i]);
    delete[] h->host_ev;
    if (h->host_in) cudaStreamDestroy(h->host_in);
    if (h->host_out) cudaStreamDestroy(h->host_out);
    delete h;
    return LOCOCO_OK;
}

lococo_status lococo_workspace_bytes(const lococo_handle* h, size_t* out) {
    if (!h || !out) return LOCOCO_ERR_INVALID_ARG;
    *out = h->ws_need;
    return LOCOCO_OK;
}

lococo_status lococo_set_workspace(lococo_handle* h, void* ptr, size_t bytes, void* stream) {
    if (!h || !ptr) return LOCOCO_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(ptr) & 255u) return LOCOCO_ERR_INVALID_ARG;
    if (bytes < h->ws_need) return LOCOCO_ERR_WORKSPACE;
    drop_loop_graph(h);
    h->ws = static_cast<char*>(ptr);
    h->weights_set = false;
    if (cudaMemsetAsync(h->ws + h->off_status, 0, 256, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return LOCOCO_ERR_CUDA;
    // The counts of the in-kernel merge (arrived CTAs, stored partial sets per unit and slot block) start at zero and
    // every step puts them back to zero. Only a kernel that gave up on an expired wait can leave them otherwise; the
    // status word then stays set as well, and both are cleared by handing the workspace over again.
    if (h->use_tensor && cudaMemsetAsync(h->ws + h->off_merge, 0, (size_t)h->units * (h->cfg.M / 128) * 2 * sizeof(int),
                                         static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return LOCOCO_ERR_CUDA;
    return LOCOCO_OK;
}

lococo_status lococo_set_protected_slots(lococo_handle* h, int32_t slots) {
    if (!h || slots < 0 || slots > h->cfg.M) return LOCOCO_ERR_INVALID_ARG;
    if (slots != h->prot) drop_loop_graph(h);   // a cached chunk loop carries the old count in its launches
    h->prot = slots;
    return LOCOCO_OK;
}

lococo_status lococo_set_weights(lococo_handle* h, const void* G, const void* bias, void* stream) {
    if (!h || !G || !aligned16(G)) return LOCOCO_ERR_INVALID_ARG;
    if (!h->ws) return LOCOCO_ERR_WORKSPACE;
    const lococo_config& c = h->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int sets = c.weights_per_head ? c.heads : 1;
    lococo_status s = count(h, simt_pack_weights(c.dtype, G, h->ws + h->off_gpack, sets, c.M, c.c_in, c.k, st));
    if (s) return s;
    drop_loop_graph(h);
    h->has_bias = bias != nullptr;
    if (bias) {
        s = count(h, simt_convert_bias(c.dtype, bias, reinterpret_cast<float*>(h->ws + h->off_bias), sets * c.M, st));
        if (s) return s;
    }
    if (h->use_tensor) {
        s = count(h, tensor_pack_weights(h, G, st));
        if (s) return s;
    }
    h->weights_set = true;
    return LOCOCO_OK;
}

lococo_status lococo_compress_step(lococo_handle* h, lococo_tensor K_cache, lococo_tensor V_cache, int32_t cache_len,
                                   lococo_tensor K_chunk, lococo_tensor V_chunk, int32_t b, lococo_tensor K_out,
                                   lococo_tensor V_out, int32_t* new_len, float* W_out, void* stream) {
    lococo_status s = ready(h);
    if (s) return s;
    if (!chunk_args_ok(h, cache_len, b)) return LOCOCO_ERR_INVALID_ARG;
    const size_t e = h->elt;
    if (!view_ok(K_cache, e) || !view_ok(V_cache, e) || !view_ok(K_chunk, e) || !view_ok(V_chunk, e) ||
        !view_ok(K_out, e) || !view_ok(V_out, e))
        return LOCOCO_ERR_INVALID_ARG;
    if (K_out.ptr == K_chunk.ptr || V_out.ptr == V_chunk.ptr || K_out.ptr == V_out.ptr || K_out.ptr == V_cache.ptr ||
        V_out.ptr == K_cache.ptr)
        return LOCOCO_ERR_INVALID_ARG;
    if (W_out && !aligned16(W_out)) return LOCOCO_ERR_INVALID_ARG;
    s = compress_impl(h, dev(K_cache), dev(V_cache), cache_len, dev(K_chunk), dev(V_chunk), b, dev(K_out), dev(V_out),
                      cache_len + b <= h->cfg.M ? nullptr : W_out, static_cast<cudaStream_t>(stream));
    if (s) return s;
    if (new_len) *new_len = cache_len + b <= h->cfg.M ? cache_len + b : h->cfg.M;
    return LOCOCO_OK;
}

lococo_status lococo_chunk_attention(lococo_handle* h, lococo_tensor Q, lococo_tensor K_cache, lococo_tensor V_cache,
                                     int32_t cache_len, lococo_tensor K_chunk, lococo_tensor V_chunk, int32_t b,
                                     lococo_tensor O, float* lse, void* stream) {
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    if (!chunk_args_ok(h, cache_len, b)) return LOCOCO_ERR_INVALID_ARG;
    const size_t e = h->elt;
    if (!view_ok(Q, e) || !view_ok(K_chunk, e) || !view_ok(V_chunk, e) || !view_ok(O, e)) return LOCOCO_ERR_INVALID_ARG;
    if (cache_len > 0 && (!view_ok(K_cache, e) || !view_ok(V_cache, e))) return LOCOCO_ERR_INVALID_ARG;
    if (O.ptr == Q.ptr || O.ptr == K_chunk.ptr || O.ptr == V_chunk.ptr || O.ptr == K_cache.ptr || O.ptr == V_cache.ptr)
        return LOCOCO_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return LOCOCO_ERR_INVALID_ARG;
    return attention_impl(h, dev(Q), dev(K_cache), dev(V_cache), cache_len, dev(K_chunk), dev(V_chunk), b, dev(O), lse, b,
                          static_cast<cudaStream_t>(stream));
}

lococo_status lococo_saved_bytes(const lococo_handle* h, int32_t L, int32_t B, size_t* out) {
    if (!h || !out || L < 1 || B < 1) return LOCOCO_ERR_INVALID_ARG;
    const size_t n_chunks = ((size_t)L + B - 1) / B;
    const size_t snap = align_up(n_chunks * h->units * h->cfg.M * h->cfg.head_dim * h->elt, 256);
    *out = 2 * snap + align_up((size_t)h->units * L * sizeof(float), 256);
    return LOCOCO_OK;
}

}  // extern "C"

namespace {
// Algorithm 2's loop as stream-ordered launches.
lococo_status run_chunk_loop(lococo_handle* h, lococo_tensor Q, lococo_tensor K, lococo_tensor V, int32_t L, int32_t B,
                             lococo_tensor O, lococo_tensor K_cache, lococo_tensor V_cache, int* c_inout, void* saved,
                             cudaStream_t st) {
    const lococo_config& cfg = h->cfg;
    const size_t e = h->elt;
    int c = *c_inout;
    h->seq_count = 0;   // nothing is left queued from a call that failed half-way
    h->chain_open = false;
    const int n_chunks = (L + B - 1) / B;
    const size_t snap_step = (size_t)h->units * cfg.M * cfg.head_dim * e;
    const size_t snap_all = align_up((size_t)n_chunks * snap_step, 256);
    char* sv = static_cast<char*>(saved);
    // The cache the next step reads: the caller's, or (tensor-core path, while steps can write their
    // result directly) the workspace's second cache; the two alternate, so a step never writes the cache
    // its own attention CTAs are reading. The final cache is always handed back in the caller's tensors.
    View cur_k = dev(K_cache), cur_v = dev(V_cache);
    const lococo_tensor alt_k_t = contiguous(h->ws + h->off_alt_k, cfg.heads, cfg.M, cfg.head_dim);
    const lococo_tensor alt_v_t = contiguous(h->ws + h->off_alt_v, cfg.heads, cfg.M, cfg.head_dim);
    bool in_alt = false;
    for (int n = 0; n < n_chunks; ++n) {
        const int t0 = n * B;
        const int b = L - t0 < B ? L - t0 : B;
        if (sv) {
            lococo_tensor sk = contiguous(sv + (size_t)n * snap_step, cfg.heads, cfg.M, cfg.head_dim);
            lococo_tensor svv = contiguous(sv + snap_all + (size_t)n * snap_step, cfg.heads, cfg.M, cfg.head_dim);
            FillParams f{cur_k, cur_v, dev(sk), dev(svv), cfg.heads, h->units, cfg.head_dim, 0, cfg.M};
            lococo_status s = count(h, simt_fill(cfg.dtype, f, st));
            if (s) return s;
        }
        View qn = offset_tokens(Q, t0, e), kn = offset_tokens(K, t0, e), vn = offset_tokens(V, t0, e);
        View on = offset_tokens(O, t0, e);
        float* lse = sv ? reinterpret_cast<float*>(sv + 2 * snap_all) + t0 : nullptr;
        // on request, consecutive compress steps are queued for ONE persistent launch
        // (not while snapshots for a backward pass are wanted: they are taken between the steps)
        bool queued = false;
        if (h->persistent_loop && !sv && c + b > cfg.M) {
            const AttnParams a = make_attn_params(h, qn, dev(K_cache), dev(V_cache), c, kn, vn, b, on, nullptr, L);
            const CompressParams p = make_compress_params(h, dev(K_cache), dev(V_cache), c, kn, vn, b, dev(K_cache), dev(V_cache), nullptr);
            queued = tensor_attention_supported(h, a) && tensor_compress_supported(h, p) && tensor_sequence_add(h, a, p, st);
        }
        if (!queued) {
            lococo_status s = count(h, tensor_sequence_launch(h, st, h->prof.on ? &h->prof : nullptr));   // flush what is queued, in order
            if (s) return s;
            View out_k = cur_k, out_v = cur_v;
            bool direct = false;
            if (h->use_tensor && !h->persistent_loop && c + b > cfg.M) {
                const CompressParams p = make_compress_params(h, cur_k, cur_v, c, kn, vn, b, cur_k, cur_v, nullptr);
                direct = tensor_compress_supported(h, p) && tensor_step_direct(h, p);
            }
            if (direct) {
                out_k = in_alt ? dev(K_cache) : dev(alt_k_t);
                out_v = in_alt ? dev(V_cache) : dev(alt_v_t);
            }
            s = step_impl(h, qn, cur_k, cur_v, c, kn, vn, b, on, lse, L, out_k, out_v, st);
            if (s) return s;
            if (direct) {
                cur_k = out_k;
                cur_v = out_v;
                in_alt = !in_alt;
            }
        }
        c = c + b <= cfg.M ? c + b : cfg.M;
    }
    lococo_status s = count(h, tensor_sequence_launch(h, st, h->prof.on ? &h->prof : nullptr));
    if (s) return s;
    if (in_alt) {   // hand the final cache back
        FillParams f{cur_k, cur_v, dev(K_cache), dev(V_cache), cfg.heads, h->units, cfg.head_dim, 0, cfg.M};
        s = count(h, simt_fill(cfg.dtype, f, st));
        if (s) return s;
    }
    *c_inout = c;
    return LOCOCO_OK;
}
}  // namespace

extern "C" {
lococo_status lococo_process_sequence(lococo_handle* h, lococo_tensor Q, lococo_tensor K, lococo_tensor V, int32_t L,
                                      int32_t B, lococo_tensor O, lococo_tensor K_cache, lococo_tensor V_cache,
                                      int32_t* cache_len_inout, void* saved, void* stream) {
    lococo_status s = ready(h);
    if (s) return s;
    if (!cache_len_inout || L < 1 || B < 1 || B > h->cfg.max_chunk) return LOCOCO_ERR_INVALID_ARG;
    int c = *cache_len_inout;
    if (c < 0 || c > h->cfg.M) return LOCOCO_ERR_INVALID_ARG;
    const size_t e = h->elt;
    if (!view_ok(Q, e) || !view_ok(K, e) || !view_ok(V, e) || !view_ok(O, e) || !view_ok(K_cache, e) || !view_ok(V_cache, e))
        return LOCOCO_ERR_INVALID_ARG;
    if (O.ptr == Q.ptr || O.ptr == K.ptr || O.ptr == V.ptr || K_cache.ptr == V_cache.ptr) return LOCOCO_ERR_INVALID_ARG;
    if (saved && (reinterpret_cast<uintptr_t>(saved) & 255u)) return LOCOCO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int c_in = c;

    // The loop is a fixed sequence of launches for a given argument set, so repeated calls with the
    // same arguments (a serving loop over one set of buffers) replay it as a CUDA graph: kernel-to-
    // kernel hand-over inside a graph is shorter than between stream launches. First call: eager.
    // Second identical call: captured, instantiated, launched. Later calls: graph launch only.
    lococo_handle::LoopGraph& lg = h->loop_graph;
    struct Key { lococo_tensor Q, K, V, O, Kc, Vc; void* saved; int32_t L, B, c, pad; } key;
    std::memset(&key, 0, sizeof(key));   // padding bytes take part in the comparison
    key.Q = Q; key.K = K; key.V = V; key.O = O; key.Kc = K_cache; key.Vc = V_cache;
    key.saved = saved; key.L = L; key.B = B; key.c = c_in;
    static_assert(sizeof(key) <= sizeof(lg.key), "key buffer too small");
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    // (the legacy default stream cannot be captured: callers on it always get the eager loop)
    // (nor is the persistent loop captured: its step descriptors reach the device by a copy from a small ring of pinned
    // host slots that later eager calls reuse, so a replay would read whatever the ring holds by then)
    const bool graph_ok = !lg.disabled && !h->prof.on && h->use_tensor && !h->persistent_loop && st != nullptr && st != cudaStreamLegacy &&
                          st != cudaStreamPerThread && cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
    const bool same = graph_ok && lg.key_len == sizeof(key) && std::memcmp(lg.key, &key, sizeof(key)) == 0;
    if (same && lg.exec) {
        if (cudaGraphLaunch(lg.exec, st) == cudaSuccess) {
            h->launches += lg.launches;
            *cache_len_inout = lg.c_out;
            return LOCOCO_OK;
        }
        lg.disabled = true;
    }
    if (graph_ok && !same) {
        if (lg.exec) { cudaGraphExecDestroy(lg.exec); lg.exec = nullptr; }
        std::memset(lg.key, 0, sizeof(lg.key));
        std::memcpy(lg.key, &key, sizeof(key));
        lg.key_len = sizeof(key);
        lg.seen = 0;
    }
    const bool capture = graph_ok && same && !lg.disabled && lg.seen >= 1 && !lg.exec;
    if (graph_ok) ++lg.seen;
    if (capture && cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        lg.disabled = true;
        cudaGetLastError();   // clear the refusal so that it is not mistaken for a launch failure
        return lococo_process_sequence(h, Q, K, V, L, B, O, K_cache, V_cache, cache_len_inout, saved, stream);
    }
    const int64_t launches_before = h->launches;
    s = run_chunk_loop(h, Q, K, V, L, B, O, K_cache, V_cache, &c, saved, st);
    if (capture) {
        cudaGraph_t graph = nullptr;
        const bool ended = cudaStreamEndCapture(st, &graph) == cudaSuccess && graph != nullptr;
        bool launched = false;
        if (ended && s == LOCOCO_OK && cudaGraphInstantiate(&lg.exec, graph, 0) == cudaSuccess) {
            lg.launches = h->launches - launches_before;
            lg.c_out = c;
            launched = cudaGraphLaunch(lg.exec, st) == cudaSuccess;
        }
        if (graph) cudaGraphDestroy(graph);
        if (!launched) {
            // nothing has run yet (the launches were only recorded): fall back to the eager loop
            if (lg.exec) { cudaGraphExecDestroy(lg.exec); lg.exec = nullptr; }
            lg.disabled = true;
            cudaGetLastError();
            h->launches = launches_before;
            c = c_in;
            s = run_chunk_loop(h, Q, K, V, L, B, O, K_cache, V_cache, &c, saved, st);
        }
    }
    if (s) return s;
    *cache_len_inout = c;
    return LOCOCO_OK;
}

lococo_status lococo_host_staging_bytes(const lococo_handle* h, int32_t L, size_t* out) {
    if (!h || !out || L < 1) return LOCOCO_ERR_INVALID_ARG;
    const size_t seq = align_up((size_t)h->units * L * h->cfg.head_dim * h->elt, 256);
    const size_t cache = align_up((size_t)h->units * h->cfg.M * h->cfg.head_dim * h->elt, 256);
    *out = 4 * seq + 2 * cache;
    return LOCOCO_OK;
}

lococo_status lococo_process_sequence_host(lococo_handle* h, const void* Qh, const void* Kh, const void* Vh, int32_t L,
                                           int32_t B, void* Oh, void* Kc_h, void* Vc_h, int32_t* final_len,
                                           void* staging, size_t staging_bytes, void* stream) {
    if (!h || !Qh || !Kh || !Vh || !Oh || !staging || L < 1) return LOCOCO_ERR_INVALID_ARG;
    if (B < 1 || B > h->cfg.max_chunk) return LOCOCO_ERR_INVALID_ARG;   // the scratch is sized for chunks of at most max_chunk
    lococo_status s = ready(h);
    if (s) return s;
    if (reinterpret_cast<uintptr_t>(staging) & 255u) return LOCOCO_ERR_INVALID_ARG;
    size_t need = 0;
    lococo_host_staging_bytes(h, L, &need);
    if (staging_bytes < need) return LOCOCO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const lococo_config& cfg = h->cfg;
    const size_t seq_bytes = (size_t)h->units * L * cfg.head_dim * h->elt;
    const size_t seq = align_up(seq_bytes, 256);
    const size_t cache_bytes = (size_t)h->units * cfg.M * cfg.head_dim * h->elt;
    const size_t cache = align_up(cache_bytes, 256);
    char* base = static_cast<char*>(staging);
    char *dQ = base, *dK = base + seq, *dV = base + 2 * seq, *dO = base + 3 * seq;
    char *dKc = base + 4 * seq, *dVc = dKc + cache;
    // Chunk by chunk on three streams: the copy of chunk n+1 to the device, the step of chunk n
    // (Algorithm 2 needs nothing beyond chunk n and the cache) and the copy of chunk n-1's output back
    // run at the same time, so the call costs about as much as its longest leg (normally the inputs).
    const int n_chunks = (L + B - 1) / B;
    if (!h->host_in && (cudaStreamCreateWithFlags(&h->host_in, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaStreamCreateWithFlags(&h->host_out, cudaStreamNonBlocking) != cudaSuccess))
        return LOCOCO_ERR_CUDA;
    if (h->host_ev_n < 2 * n_chunks + 2) {
        cudaEvent_t* ev = new (std::nothrow) cudaEvent_t[2 * n_chunks + 2]();
        if (!ev) return LOCOCO_ERR_CUDA;
        for (int i = 0; i < h->host_ev_n; ++i) ev[i] = h->host_ev[i];
        for (int i = h->host_ev_n; i < 2 * n_chunks + 2; ++i)
            if (cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) != cudaSuccess) {
                for (int j = h->host_ev_n; j < i; ++j) cudaEventDestroy(ev[j]);
                delete[] ev;
                return LOCOCO_ERR_CUDA;
            }
        delete[] h->host_ev;
        h->host_ev = ev;
        h->host_ev_n = 2 * n_chunks + 2;
    }
    cudaEvent_t* ev_in = h->host_ev;                 // chunk n is on the device
    cudaEvent_t* ev_done = h->host_ev + n_chunks;    // chunk n's output is complete
    cudaEvent_t ev_start = h->host_ev[2 * n_chunks], ev_out = h->host_ev[2 * n_chunks + 1];
    const size_t row = (size_t)cfg.head_dim * h->elt, pitch = (size_t)L * row;
    // the staging area is free once the work already queued on `stream` is done
    if (cudaEventRecord(ev_start, st) != cudaSuccess || cudaStreamWaitEvent(h->host_in, ev_start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(h->host_out, ev_start, 0) != cudaSuccess)
        return LOCOCO_ERR_CUDA;
    for (int n = 0; n < n_chunks; ++n) {
        const size_t off = (size_t)n * B * row;
        const size_t width = (size_t)std::min(B, L - n * B) * row;
        if (cudaMemcpy2DAsync(dQ + off, pitch, static_cast<const char*>(Qh) + off, pitch, width, h->units, cudaMemcpyHostToDevice, h->host_in) != cudaSuccess ||
            cudaMemcpy2DAsync(dK + off, pitch, static_cast<const char*>(Kh) + off, pitch, width, h->units, cudaMemcpyHostToDevice, h->host_in) != cudaSuccess ||
            cudaMemcpy2DAsync(dV + off, pitch, static_cast<const char*>(Vh) + off, pitch, width, h->units, cudaMemcpyHostToDevice, h->host_in) != cudaSuccess ||
            cudaEventRecord(ev_in[n], h->host_in) != cudaSuccess)
            return LOCOCO_ERR_CUDA;
    }
    int c = 0;
    const lococo_tensor tQ = contiguous(dQ, cfg.heads, L, cfg.head_dim), tK = contiguous(dK, cfg.heads, L, cfg.head_dim);
    const lococo_tensor tV = contiguous(dV, cfg.heads, L, cfg.head_dim), tO = contiguous(dO, cfg.heads, L, cfg.head_dim);
    const lococo_tensor tKc = contiguous(dKc, cfg.heads, cfg.M, cfg.head_dim), tVc = contiguous(dVc, cfg.heads, cfg.M, cfg.head_dim);
    for (int n = 0; n < n_chunks; ++n) {
        const int t0 = n * B, b = std::min(B, L - t0);
        const size_t off = (size_t)t0 * row;
        if (cudaStreamWaitEvent(st, ev_in[n], 0) != cudaSuccess) return LOCOCO_ERR_CUDA;
        auto from = [&](lococo_tensor t) {
            t.ptr = static_cast<char*>(t.ptr) + off;
            return t;
        };
        s = run_chunk_loop(h, from(tQ), from(tK), from(tV), b, B, from(tO), tKc, tVc, &c, nullptr, st);
        if (s) return s;
        if (cudaEventRecord(ev_done[n], st) != cudaSuccess || cudaStreamWaitEvent(h->host_out, ev_done[n], 0) != cudaSuccess ||
            cudaMemcpy2DAsync(static_cast<char*>(Oh) + off, pitch, dO + off, pitch, (size_t)b * row, h->units, cudaMemcpyDeviceToHost, h->host_out) != cudaSuccess)
            return LOCOCO_ERR_CUDA;
    }
    if (cudaEventRecord(ev_out, h->host_out) != cudaSuccess || cudaStreamWaitEvent(st, ev_out, 0) != cudaSuccess) return LOCOCO_ERR_CUDA;
    if (Kc_h && cudaMemcpyAsync(Kc_h, dKc, cache_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return LOCOCO_ERR_CUDA;
    if (Vc_h && cudaMemcpyAsync(Vc_h, dVc, cache_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return LOCOCO_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LOCOCO_ERR_CUDA;
    if (final_len) *final_len = c;
    return LOCOCO_OK;
}

lococo_status lococo_get_last_device_status(lococo_handle* h, int32_t* out, void* stream) {
    if (!h || !out) return LOCOCO_ERR_INVALID_ARG;
    if (!h->ws) return LOCOCO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, h->ws + h->off_status, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return LOCOCO_ERR_CUDA;
    *out = word == 0 ? LOCOCO_OK : LOCOCO_ERR_TIMEOUT;
    return LOCOCO_OK;
}

lococo_status lococo_launch_count(const lococo_handle* h, int64_t* out) {
    if (!h || !out) return LOCOCO_ERR_INVALID_ARG;
    *out = h->launches;
    return LOCOCO_OK;
}

}  // extern "C"
