// lococo_compress_step_static: the compress step for callers that cannot allocate device
// memory. Its scratch lives in a fixed array inside the library image instead of a
// caller-provided workspace.
#include <atomic>

#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;  // 8 MiB, resident on every GPU that loads the library

// Device-side storage. In host code this name is only a handle for the runtime's symbol
// table, never an address a kernel may be given: the device address is looked up below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<unsigned char*> g_scratch_addr[kMaxDevices];

// Device address of the array on the current device; looked up once per device. Host threads that make
// their first call at the same time each run the query and store the same address.
unsigned char* scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    unsigned char* ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess) return nullptr;
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

bool view_ok(const lococo_tensor& t, size_t elt) {
    if (!t.ptr || (reinterpret_cast<uintptr_t>(t.ptr) & 15u)) return false;
    if ((t.stride_batch * (int64_t)elt) % 16 || (t.stride_head * (int64_t)elt) % 16 || (t.stride_token * (int64_t)elt) % 16)
        return false;
    return t.stride_token > 0;
}

lococo::View dev(const lococo_tensor& t) {
    return lococo::View{static_cast<char*>(t.ptr), t.stride_batch, t.stride_head, t.stride_token};
}

}  // namespace

extern "C" {

lococo_status lococo_static_scratch_limit(size_t* out) {
    if (!out) return LOCOCO_ERR_INVALID_ARG;
    *out = kStaticScratchBytes;
    return LOCOCO_OK;
}

lococo_status lococo_compress_step_static(const lococo_config* cfg, const void* G, const void* bias,
                                          lococo_tensor K_cache, lococo_tensor V_cache, int32_t cache_len,
                                          lococo_tensor K_chunk, lococo_tensor V_chunk, int32_t b,
                                          lococo_tensor K_out, lococo_tensor V_out, void* stream) {
    using namespace lococo;
    if (!cfg || !G || (reinterpret_cast<uintptr_t>(G) & 15u)) return LOCOCO_ERR_INVALID_ARG;
    const lococo_config& c = *cfg;
    if (c.batch < 1 || c.heads < 1 || c.M < 1 || c.k < 1 || c.k % 2 == 0) return LOCOCO_ERR_INVALID_ARG;
    if (c.dtype != LOCOCO_F32 && c.dtype != LOCOCO_BF16) return LOCOCO_ERR_INVALID_ARG;
    if (c.c_in != c.head_dim && c.c_in != 2 * c.head_dim) return LOCOCO_ERR_INVALID_ARG;
    if (c.weights_per_head != 0 && c.weights_per_head != 1) return LOCOCO_ERR_INVALID_ARG;
    if (!(c.norm_eps >= 0.f)) return LOCOCO_ERR_INVALID_ARG;
    if ((c.head_dim != 64 && c.head_dim != 128) || c.k > 63 || (int64_t)c.batch * c.heads > 65535)
        return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    if (cache_len < 0 || cache_len > c.M || b < 1) return LOCOCO_ERR_INVALID_ARG;
    if ((int64_t)cache_len + b <= c.M) return LOCOCO_ERR_INVALID_ARG;  // the fill branch needs no scratch: use lococo_compress_step
    const size_t e = c.dtype == LOCOCO_F32 ? 4 : 2;
    if (!view_ok(K_cache, e) || !view_ok(V_cache, e) || !view_ok(K_chunk, e) || !view_ok(V_chunk, e) ||
        !view_ok(K_out, e) || !view_ok(V_out, e))
        return LOCOCO_ERR_INVALID_ARG;
    if (K_out.ptr == K_chunk.ptr || V_out.ptr == V_chunk.ptr || K_out.ptr == V_out.ptr || K_out.ptr == V_cache.ptr ||
        V_out.ptr == K_cache.ptr)
        return LOCOCO_ERR_INVALID_ARG;

    // scratch layout: packed weights | bias as fp32 | row sums | both blends | ReLU'd logits
    const size_t units = (size_t)c.batch * c.heads, sets = c.weights_per_head ? c.heads : 1;
    const size_t S = (size_t)cache_len + b;
    size_t off = 0;
    const size_t off_g = off;    off = align256(off + sets * c.k * c.M * c.c_in * e);
    const size_t off_bias = off; off = align256(off + sets * c.M * sizeof(float));
    const size_t off_s = off;    off = align256(off + units * c.M * sizeof(float));
    const size_t off_uk = off;   off = align256(off + units * c.M * c.head_dim * sizeof(float));
    const size_t off_uv = off;   off = align256(off + units * c.M * c.head_dim * sizeof(float));
    const size_t off_r = off;    off = align256(off + units * c.M * S * sizeof(float));
    if (off > kStaticScratchBytes) return LOCOCO_ERR_WORKSPACE;  // problem too large for the built-in scratch

    unsigned char* scratch = scratch_for_current_device();
    if (!scratch) return LOCOCO_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    if (simt_pack_weights(c.dtype, G, scratch + off_g, (int)sets, c.M, c.c_in, c.k, st) < 0) return LOCOCO_ERR_CUDA;
    if (bias && simt_convert_bias(c.dtype, bias, reinterpret_cast<float*>(scratch + off_bias), (int)sets * c.M, st) < 0)
        return LOCOCO_ERR_CUDA;
    CompressParams p{};
    p.xk = CatView{dev(K_cache), dev(K_chunk), cache_len, b};
    p.xv = CatView{dev(V_cache), dev(V_chunk), cache_len, b};
    p.k_out = dev(K_out);
    p.v_out = dev(V_out);
    p.heads = c.heads; p.units = (int)units; p.d = c.head_dim; p.M = c.M; p.k = c.k; p.c_in = c.c_in;
    p.S = (int)S;
    p.weights_per_head = c.weights_per_head;
    p.g_packed = scratch + off_g;
    p.bias = bias ? reinterpret_cast<const float*>(scratch + off_bias) : nullptr;
    p.eps = c.norm_eps;
    p.R = reinterpret_cast<float*>(scratch + off_r);
    p.s = reinterpret_cast<float*>(scratch + off_s);
    p.UK = reinterpret_cast<float*>(scratch + off_uk);
    p.UV = reinterpret_cast<float*>(scratch + off_uv);
    p.W_out = nullptr;
    p.prof = nullptr;
    return simt_compress(c.dtype, p, st) < 0 ? LOCOCO_ERR_CUDA : LOCOCO_OK;
}

}  // extern "C"
