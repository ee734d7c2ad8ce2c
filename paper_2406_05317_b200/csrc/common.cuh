// Internal declarations shared by the LoCoCo CUDA translation units.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lococo.h"

namespace lococo {

// Device-side view of a lococo_tensor (strides in elements).
struct View {
    char* ptr;
    int64_t sb, sh, st;
};

// One (sequence, head) unit's [cache; chunk] concatenation, cache first (Eq. 3).
struct CatView {
    View cache, chunk;
    int c;  // valid cache rows
    int b;  // chunk rows
};

template <typename T>
__device__ __forceinline__ const T* unit_base(const View& v, int n, int h) {
    return reinterpret_cast<const T*>(v.ptr) + n * v.sb + h * v.sh;
}
template <typename T>
__device__ __forceinline__ T* unit_base_mut(const View& v, int n, int h) {
    return reinterpret_cast<T*>(v.ptr) + n * v.sb + h * v.sh;
}
// Row j of the concatenation for unit (n, h).
template <typename T>
__device__ __forceinline__ const T* cat_row(const CatView& x, int n, int h, int j) {
    return j < x.c ? unit_base<T>(x.cache, n, h) + (int64_t)j * x.cache.st
                   : unit_base<T>(x.chunk, n, h) + (int64_t)(j - x.c) * x.chunk.st;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Parameters of one compress step (Algorithm 2, Steps 4-5) for all units.
struct CompressParams {
    CatView xk, xv;       // keys and values, [cache; chunk]
    View k_out, v_out;    // new cache
    int heads, units, d, M, k, c_in, S;
    int weights_per_head;
    const void* g_packed;  // [heads|1][k][M][c_in], storage dtype
    const float* bias;     // [heads|1][M] or nullptr
    float eps;
    float* R;              // [units][M][S] ReLU'd logits
    float* s;              // [units][M] denominators of Eq. 7
    float* UK;             // [units][M][d] unnormalised blends
    float* UV;
    float* W_out;          // optional [units][M][S]
    void* R16;             // optional bf16 copy of R, [units][M][R16_stride] (the backward's recompute; tensor-core path only)
    int R16_stride;        // multiple of 8
    int prot = 0;          // protected slots (Section 5.2): rows i < prot of Eq. 7's matrix are the unit rows e_i
    void* prof;            // host only: Profiler* or nullptr
};

// Parameters of one chunk attention (Algorithm 2, Step 3) for all units.
struct AttnParams {
    View q, o;
    CatView xk, xv;
    int heads, units, d, b, c;
    float scale;
    float* lse;        // optional [units][lse_stride]
    int64_t lse_stride;
    void* prof;        // host only: Profiler* or nullptr
};

struct FillParams {
    View src_k, src_v, dst_k, dst_v;  // src rows 0..b-1 -> dst rows c..c+b-1
    int heads, units, d, c, b;
};

// CUDA-core kernels (simt_forward.cu). Each returns the number of kernels launched, or -1.
int simt_pack_weights(int dtype, const void* G, void* packed, int sets, int M, int c_in, int k, cudaStream_t st);
int simt_fill(int dtype, const FillParams& p, cudaStream_t st);
int simt_compress(int dtype, const CompressParams& p, cudaStream_t st);
int simt_attention(int dtype, const AttnParams& p, cudaStream_t st);
// Brackets the launches between them with an event pair when p is a live Profiler*.
void prof_begin(void* p, int kind, cudaStream_t st);
void prof_end(void* p, cudaStream_t st);

int simt_convert_bias(int dtype, const void* bias, float* out, int n, cudaStream_t st);

}  // namespace lococo
