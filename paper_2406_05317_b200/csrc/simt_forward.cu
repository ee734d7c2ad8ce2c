// CUDA-core (fp32 FMA) kernels of the LoCoCo chunk step. They serve the fp32
// storage type, whose 1e-4 tolerance rules out tensor-core input rounding, and any
// shape the tensor-core kernels do not cover. Storage type T is float or bf16;
// all arithmetic is fp32.
#include "common.cuh"

namespace lococo {
namespace {

constexpr int kMaxTaps = 63;

// ------------------------------------------------------------------ weight packing
// G [sets][M][C][k]  ->  packed [sets][k][M][C]  (contraction axis contiguous per tap).
template <typename T>
__global__ void pack_weights_kernel(const T* __restrict__ G, T* __restrict__ out, int sets, int M, int C, int k) {
    const int64_t total = (int64_t)sets * M * C * k;
    for (int64_t o = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int ch = o % C;
        int64_t r = o / C;
        const int i = r % M;
        r /= M;
        const int t = r % k;
        const int set = r / k;
        out[o] = G[(((int64_t)set * M + i) * C + ch) * k + t];
    }
}

template <typename T>
__global__ void to_f32_kernel(const T* __restrict__ in, float* __restrict__ out, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = to_f32(in[i]);
}

// ------------------------------------------------------------------ fill branch
template <typename T>
__global__ void fill_kernel(FillParams p) {
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int vec = 16 / sizeof(T), per_row = p.d / vec;
    const int total = p.b * per_row;
    for (int x = blockIdx.x * blockDim.x + threadIdx.x; x < total; x += gridDim.x * blockDim.x) {
        const int r = x / per_row, v = x % per_row;
        const int4* sk = reinterpret_cast<const int4*>(unit_base<T>(p.src_k, n, h) + (int64_t)r * p.src_k.st) + v;
        const int4* sv = reinterpret_cast<const int4*>(unit_base<T>(p.src_v, n, h) + (int64_t)r * p.src_v.st) + v;
        int4* dk = reinterpret_cast<int4*>(unit_base_mut<T>(p.dst_k, n, h) + (int64_t)(p.c + r) * p.dst_k.st) + v;
        int4* dv = reinterpret_cast<int4*>(unit_base_mut<T>(p.dst_v, n, h) + (int64_t)(p.c + r) * p.dst_v.st) + v;
        *dk = *sk;
        *dv = *sv;
    }
}

// ------------------------------------------------------------------ Eq. 6 + ReLU
// R[u][i][j] = max(0, bias_i + sum_t sum_ch Gp[t][i][ch] * Z[j+t-p][ch]).
// Block: 64 slots x 64 positions, 256 threads, 4x4 outputs per thread (strided by 16).
constexpr int CT = 64;   // tile edge
constexpr int CCH = 32;  // channels per stage

template <typename T>
__global__ void __launch_bounds__(256) conv_relu_kernel(CompressParams p) {
    extern __shared__ float smem[];
    const int rows = CT + p.k - 1;
    float* Zs = smem;                      // [rows][CCH+1]
    float* Gs = smem + rows * (CCH + 1);   // [CT][CCH+1]
    const int u = blockIdx.z, n = u / p.heads, h = u % p.heads;
    const int j0 = blockIdx.x * CT, i0 = blockIdx.y * CT;
    const int pad = (p.k - 1) / 2;
    const int tid = threadIdx.x, tj = tid % 16, ti = tid / 16;
    const T* gp = reinterpret_cast<const T*>(p.g_packed) + (p.weights_per_head ? (int64_t)h * p.k * p.M * p.c_in : 0);

    float acc[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;

    for (int ch0 = 0; ch0 < p.c_in; ch0 += CCH) {
        // stage the input rows j0-pad .. j0+CT+pad-1 for channels ch0..ch0+31
        __syncthreads();
        for (int x = tid; x < rows * CCH; x += 256) {
            const int r = x / CCH, cc = x % CCH;
            const int j = j0 - pad + r, ch = ch0 + cc;
            float z = 0.f;
            if (j >= 0 && j < p.S && ch < p.c_in) {
                z = ch < p.d ? to_f32(cat_row<T>(p.xk, n, h, j)[ch]) : to_f32(cat_row<T>(p.xv, n, h, j)[ch - p.d]);
            }
            Zs[r * (CCH + 1) + cc] = z;
        }
        for (int t = 0; t < p.k; ++t) {
            __syncthreads();
            for (int x = tid; x < CT * CCH; x += 256) {
                const int r = x / CCH, cc = x % CCH;
                const int i = i0 + r, ch = ch0 + cc;
                Gs[r * (CCH + 1) + cc] = (i < p.M && ch < p.c_in) ? to_f32(gp[((int64_t)t * p.M + i) * p.c_in + ch]) : 0.f;
            }
            __syncthreads();
#pragma unroll 8
            for (int cc = 0; cc < CCH; ++cc) {
                float g[4], z[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) g[x] = Gs[(ti + 16 * x) * (CCH + 1) + cc];
#pragma unroll
                for (int y = 0; y < 4; ++y) z[y] = Zs[(tj + 16 * y + t) * (CCH + 1) + cc];
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(g[x], z[y], acc[x][y]);
            }
        }
    }
    const float* bias = p.bias ? p.bias + (p.weights_per_head ? h * p.M : 0) : nullptr;
    float* R = p.R + (int64_t)u * p.M * p.S;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int i = i0 + ti + 16 * x;
        if (i >= p.M) continue;
        const float bi = bias ? bias[i] : 0.f;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int j = j0 + tj + 16 * y;
            if (j < p.S) R[(int64_t)i * p.S + j] = i < p.prot ? (j == i ? 1.f : 0.f) : fmaxf(acc[x][y] + bi, 0.f);
        }
    }
}

// ------------------------------------------------------------------ Eq. 7 denominators
// One warp per (unit, slot) row; fixed summation order.
// A protected slot's row is a unit row and its denominator exactly 1 (no eps), so it keeps its entry bit for bit.
__global__ void rowsum_kernel(const float* __restrict__ R, float* __restrict__ s, int rows, int S, float eps, int M, int prot) {
    const int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    if (row >= rows) return;
    const int lane = threadIdx.x % 32;
    const float* r = R + (int64_t)row * S;
    float acc = 0.f;
    for (int j = lane; j < S; j += 32) acc += r[j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) s[row] = row % M < prot ? 1.f : acc + eps;
}

// ------------------------------------------------------------------ Eq. 4, Eq. 5 (unnormalised)
// UK[u][i][:] = sum_j R[u][i][j] XK[j][:], UV likewise. Block: SLOTS slots x D channels.
template <typename T, int D>
__global__ void __launch_bounds__(256) blend_kernel(CompressParams p) {
    constexpr int TX = D / 4;          // threads along channels (float4 each)
    constexpr int TY = 256 / TX;       // thread rows
    constexpr int SLOTS = TY * 4;      // slots per block
    constexpr int JT = 32;             // positions per stage
    __shared__ float Rs[SLOTS][JT + 1];
    __shared__ __align__(16) float Ks[JT][D];
    __shared__ __align__(16) float Vs[JT][D];
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int i0 = blockIdx.x * SLOTS;
    const int tid = threadIdx.x, tx = tid % TX, ty = tid / TX;
    const float* R = p.R + (int64_t)u * p.M * p.S;
    float aK[4][4], aV[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) aK[x][y] = aV[x][y] = 0.f;

    for (int j0 = 0; j0 < p.S; j0 += JT) {
        __syncthreads();
        for (int x = tid; x < SLOTS * JT; x += 256) {
            const int r = x / JT, jj = x % JT;
            const int i = i0 + r, j = j0 + jj;
            Rs[r][jj] = (i < p.M && j < p.S) ? R[(int64_t)i * p.S + j] : 0.f;
        }
        for (int x = tid; x < JT * D; x += 256) {
            const int jj = x / D, ch = x % D;
            const int j = j0 + jj;
            float kv = 0.f, vv = 0.f;
            if (j < p.S) {
                kv = to_f32(cat_row<T>(p.xk, n, h, j)[ch]);
                vv = to_f32(cat_row<T>(p.xv, n, h, j)[ch]);
            }
            Ks[jj][ch] = kv;
            Vs[jj][ch] = vv;
        }
        __syncthreads();
#pragma unroll 4
        for (int jj = 0; jj < JT; ++jj) {
            const float4 kx = *reinterpret_cast<const float4*>(&Ks[jj][tx * 4]);
            const float4 vx = *reinterpret_cast<const float4*>(&Vs[jj][tx * 4]);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float r = Rs[ty * 4 + x][jj];
                aK[x][0] = fmaf(r, kx.x, aK[x][0]); aK[x][1] = fmaf(r, kx.y, aK[x][1]);
                aK[x][2] = fmaf(r, kx.z, aK[x][2]); aK[x][3] = fmaf(r, kx.w, aK[x][3]);
                aV[x][0] = fmaf(r, vx.x, aV[x][0]); aV[x][1] = fmaf(r, vx.y, aV[x][1]);
                aV[x][2] = fmaf(r, vx.z, aV[x][2]); aV[x][3] = fmaf(r, vx.w, aV[x][3]);
            }
        }
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int i = i0 + ty * 4 + x;
        if (i >= p.M) continue;
        float* uk = p.UK + ((int64_t)u * p.M + i) * D + tx * 4;
        float* uv = p.UV + ((int64_t)u * p.M + i) * D + tx * 4;
        *reinterpret_cast<float4*>(uk) = make_float4(aK[x][0], aK[x][1], aK[x][2], aK[x][3]);
        *reinterpret_cast<float4*>(uv) = make_float4(aV[x][0], aV[x][1], aV[x][2], aV[x][3]);
    }
}

// new cache = U / s (Eq. 7 applied after the blend: the division commutes with the sum).
template <typename T>
__global__ void finalize_cache_kernel(CompressParams p) {
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int total = p.M * p.d;
    for (int x = blockIdx.x * blockDim.x + threadIdx.x; x < total; x += gridDim.x * blockDim.x) {
        const int i = x / p.d, ch = x % p.d;
        const float inv = 1.f / p.s[(int64_t)u * p.M + i];
        const int64_t src = ((int64_t)u * p.M + i) * p.d + ch;
        unit_base_mut<T>(p.k_out, n, h)[(int64_t)i * p.k_out.st + ch] = from_f32<T>(p.UK[src] * inv);
        unit_base_mut<T>(p.v_out, n, h)[(int64_t)i * p.v_out.st + ch] = from_f32<T>(p.UV[src] * inv);
    }
}

__global__ void write_weights_kernel(const float* __restrict__ R, const float* __restrict__ s, float* __restrict__ W,
                                     int64_t rows, int S) {
    const int64_t total = rows * S;
    for (int64_t x = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; x < total; x += (int64_t)gridDim.x * blockDim.x)
        W[x] = R[x] / s[x / S];
}

// ------------------------------------------------------------------ Eq. 1, chunk form
// 32 queries per block, 4 threads per query; each thread owns D/4 channels of q and of
// the output accumulator, interleaved in float4 groups so a quad reads 64 contiguous bytes.
template <typename T, int D>
__global__ void __launch_bounds__(128) attention_kernel(AttnParams p) {
    constexpr int NV = D / 16;  // float4 groups per thread
    constexpr int KT = 32;      // keys per tile
    __shared__ __align__(16) float Ks[KT][D];
    __shared__ __align__(16) float Vs[KT][D];
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int tid = threadIdx.x, m = tid % 4;
    const int r = blockIdx.x * 32 + tid / 4;  // query row in the chunk
    const bool live = r < p.b;
    const float sc = p.scale * 1.4426950408889634f;  // logits in base-2 units

    float4 q[NV], acc[NV];
    {
        const T* qrow = unit_base<T>(p.q, n, h) + (int64_t)(live ? r : 0) * p.q.st;
#pragma unroll
        for (int e = 0; e < NV; ++e) {
            const int ch = 4 * (m + 4 * e);
            q[e] = make_float4(to_f32(qrow[ch]) * sc, to_f32(qrow[ch + 1]) * sc, to_f32(qrow[ch + 2]) * sc,
                               to_f32(qrow[ch + 3]) * sc);
            acc[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    float mrun = -INFINITY, lrun = 0.f;
    const int S = p.c + p.b;
    const int last_row = min((int)blockIdx.x * 32 + 31, p.b - 1);
    const int ncols = p.c + last_row + 1;  // columns any query of this block can see
    const int my_cols = p.c + r + 1;       // columns this query sees

    for (int j0 = 0; j0 < ncols; j0 += KT) {
        __syncthreads();
        for (int x = tid; x < KT * D; x += 128) {
            const int jj = x / D, ch = x % D;
            const int j = j0 + jj;
            float kv = 0.f, vv = 0.f;
            if (j < S) {
                kv = to_f32(cat_row<T>(p.xk, n, h, j)[ch]);
                vv = to_f32(cat_row<T>(p.xv, n, h, j)[ch]);
            }
            Ks[jj][ch] = kv;
            Vs[jj][ch] = vv;
        }
        __syncthreads();
        float sv[KT];
        float tmax = -INFINITY;
#pragma unroll
        for (int jj = 0; jj < KT; ++jj) {
            float dot = 0.f;
#pragma unroll
            for (int e = 0; e < NV; ++e) {
                const float4 kx = *reinterpret_cast<const float4*>(&Ks[jj][4 * (m + 4 * e)]);
                dot = fmaf(q[e].x, kx.x, dot); dot = fmaf(q[e].y, kx.y, dot);
                dot = fmaf(q[e].z, kx.z, dot); dot = fmaf(q[e].w, kx.w, dot);
            }
            dot += __shfl_xor_sync(0xffffffffu, dot, 1);
            dot += __shfl_xor_sync(0xffffffffu, dot, 2);
            sv[jj] = (live && j0 + jj < my_cols) ? dot : -INFINITY;
            tmax = fmaxf(tmax, sv[jj]);
        }
        const float mnew = fmaxf(mrun, tmax);
        if (mnew > -INFINITY) {
            const float corr = exp2f(mrun - mnew);  // mrun = -inf on first use gives 0
            lrun *= corr;
#pragma unroll
            for (int e = 0; e < NV; ++e) { acc[e].x *= corr; acc[e].y *= corr; acc[e].z *= corr; acc[e].w *= corr; }
#pragma unroll
            for (int jj = 0; jj < KT; ++jj) {
                const float pj = exp2f(sv[jj] - mnew);
                lrun += pj;
#pragma unroll
                for (int e = 0; e < NV; ++e) {
                    const float4 vx = *reinterpret_cast<const float4*>(&Vs[jj][4 * (m + 4 * e)]);
                    acc[e].x = fmaf(pj, vx.x, acc[e].x); acc[e].y = fmaf(pj, vx.y, acc[e].y);
                    acc[e].z = fmaf(pj, vx.z, acc[e].z); acc[e].w = fmaf(pj, vx.w, acc[e].w);
                }
            }
            mrun = mnew;
        }
    }
    if (!live) return;
    const float inv = 1.f / lrun;
    T* orow = unit_base_mut<T>(p.o, n, h) + (int64_t)r * p.o.st;
#pragma unroll
    for (int e = 0; e < NV; ++e) {
        const int ch = 4 * (m + 4 * e);
        orow[ch] = from_f32<T>(acc[e].x * inv);
        orow[ch + 1] = from_f32<T>(acc[e].y * inv);
        orow[ch + 2] = from_f32<T>(acc[e].z * inv);
        orow[ch + 3] = from_f32<T>(acc[e].w * inv);
    }
    if (p.lse && m == 0) p.lse[(int64_t)u * p.lse_stride + r] = (mrun + log2f(lrun)) * 0.6931471805599453f;
}

template <typename F>
int checked(F&& launch) {
    launch();
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace

// ------------------------------------------------------------------ host launchers
int simt_pack_weights(int dtype, const void* G, void* packed, int sets, int M, int c_in, int k, cudaStream_t st) {
    const int64_t total = (int64_t)sets * M * c_in * k;
    const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
    if (dtype == LOCOCO_F32)
        return checked([&] { pack_weights_kernel<float><<<blocks, 256, 0, st>>>((const float*)G, (float*)packed, sets, M, c_in, k); });
    return checked([&] {
        pack_weights_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)G, (__nv_bfloat16*)packed, sets, M, c_in, k);
    });
}

int simt_convert_bias(int dtype, const void* bias, float* out, int n, cudaStream_t st) {
    const int blocks = (n + 255) / 256;
    if (dtype == LOCOCO_F32) return checked([&] { to_f32_kernel<float><<<blocks, 256, 0, st>>>((const float*)bias, out, n); });
    return checked([&] { to_f32_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)bias, out, n); });
}

int simt_fill(int dtype, const FillParams& p, cudaStream_t st) {
    const int vec = dtype == LOCOCO_F32 ? 4 : 8;
    const int total = p.b * (p.d / vec);
    dim3 grid((total + 255) / 256, p.units);
    if (dtype == LOCOCO_F32) return checked([&] { fill_kernel<float><<<grid, 256, 0, st>>>(p); });
    return checked([&] { fill_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(p); });
}

template <typename T>
static int compress_typed(const CompressParams& p, cudaStream_t st) {
    if (p.k > kMaxTaps) return -1;
    int launches = 0;
    {
        dim3 grid((p.S + CT - 1) / CT, (p.M + CT - 1) / CT, p.units);
        const size_t smem = sizeof(float) * ((size_t)(CT + p.k - 1) * (CCH + 1) + (size_t)CT * (CCH + 1));
        prof_begin(p.prof, 0, st);
        const int rc = checked([&] { conv_relu_kernel<T><<<grid, 256, smem, st>>>(p); });
        prof_end(p.prof, st);
        if (rc < 0) return -1;
        ++launches;
    }
    {
        const int rows = p.units * p.M;
        if (checked([&] { rowsum_kernel<<<(rows + 7) / 8, 256, 0, st>>>(p.R, p.s, rows, p.S, p.eps, p.M, p.prot); }) < 0) return -1;
        ++launches;
    }
    if (p.d == 128) {
        dim3 grid((p.M + 31) / 32, p.units);
        if (checked([&] { blend_kernel<T, 128><<<grid, 256, 0, st>>>(p); }) < 0) return -1;
    } else {
        dim3 grid((p.M + 63) / 64, p.units);
        if (checked([&] { blend_kernel<T, 64><<<grid, 256, 0, st>>>(p); }) < 0) return -1;
    }
    ++launches;
    {
        dim3 grid((p.M * p.d + 255) / 256, p.units);
        if (checked([&] { finalize_cache_kernel<T><<<grid, 256, 0, st>>>(p); }) < 0) return -1;
        ++launches;
    }
    if (p.W_out) {
        const int64_t rows = (int64_t)p.units * p.M;
        const int64_t total = rows * p.S;
        const int blocks = (int)((total + 255) / 256 < 8192 ? (total + 255) / 256 : 8192);
        if (checked([&] { write_weights_kernel<<<blocks, 256, 0, st>>>(p.R, p.s, p.W_out, rows, p.S); }) < 0) return -1;
        ++launches;
    }
    return launches;
}

// Eq. 6 + ReLU and the denominators of Eq. 7 only (the backward pass recomputes them).
int simt_conv_rowsum(int dtype, const CompressParams& p, cudaStream_t st) {
    if (p.k > kMaxTaps) return -1;
    dim3 grid((p.S + CT - 1) / CT, (p.M + CT - 1) / CT, p.units);
    const size_t smem = sizeof(float) * ((size_t)(CT + p.k - 1) * (CCH + 1) + (size_t)CT * (CCH + 1));
    const int rc = dtype == LOCOCO_F32 ? checked([&] { conv_relu_kernel<float><<<grid, 256, smem, st>>>(p); })
                                       : checked([&] { conv_relu_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(p); });
    if (rc < 0) return -1;
    const int rows = p.units * p.M;
    if (checked([&] { rowsum_kernel<<<(rows + 7) / 8, 256, 0, st>>>(p.R, p.s, rows, p.S, p.eps, p.M, p.prot); }) < 0) return -1;
    return 2;
}

int simt_write_weights(const float* R, const float* s, float* W, int64_t rows, int S, cudaStream_t st) {
    const int64_t total = rows * S;
    const int blocks = (int)((total + 255) / 256 < 8192 ? (total + 255) / 256 : 8192);
    return checked([&] { write_weights_kernel<<<blocks, 256, 0, st>>>(R, s, W, rows, S); });
}

int simt_compress(int dtype, const CompressParams& p, cudaStream_t st) {
    return dtype == LOCOCO_F32 ? compress_typed<float>(p, st) : compress_typed<__nv_bfloat16>(p, st);
}

template <typename T>
static int attention_typed(const AttnParams& p, cudaStream_t st) {
    dim3 grid((p.b + 31) / 32, p.units);
    prof_begin(p.prof, 1, st);
    const int rc = p.d == 128 ? checked([&] { attention_kernel<T, 128><<<grid, 128, 0, st>>>(p); })
                              : checked([&] { attention_kernel<T, 64><<<grid, 128, 0, st>>>(p); });
    prof_end(p.prof, st);
    return rc;
}

int simt_attention(int dtype, const AttnParams& p, cudaStream_t st) {
    return dtype == LOCOCO_F32 ? attention_typed<float>(p, st) : attention_typed<__nv_bfloat16>(p, st);
}

}  // namespace lococo
