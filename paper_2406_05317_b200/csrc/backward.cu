// Backward pass of Algorithm 2: gradients of
//   loss = <dO, O> + <dK_cache_final, K_cache_final> + <dV_cache_final, V_cache_final>
// w.r.t. Q, K, V and the conv weights (Section 3.2.1: the conv parameters are trained end to
// end), by reversing the chunk loop. Per step, with X = [cache before the step; chunk]:
//   cache update  fill:      dX[0:S]  = g                       (g = gradient w.r.t. the cache after the step)
//                 compress:  R, s recomputed from the saved cache (Eq. 6, ReLU, Eq. 7)
//                            dw  = g_K X_K^T + g_V X_V^T         (through Eq. 4, Eq. 5)
//                            dX += w^T g                          (the blend's own inputs)
//                            dA  = [A>0] (dw - <dw, w>_row) / s   (through Eq. 7 and the ReLU)
//                            dG += dA (*) Z,  dZ += dA (*) G      (through Eq. 6; dZ lands in dX)
//   attention     textbook softmax-attention gradient from dO, O and the saved log-sum-exp (Eq. 1)
//   split         first c rows of dX are the gradient w.r.t. the previous cache, the rest is dK_n, dV_n
// All arithmetic is fp32 on CUDA cores; storage type T is float or bf16.
#include <algorithm>

#include "backward.h"
#include "handle.h"

namespace lococo {

int simt_conv_rowsum(int dtype, const CompressParams& p, cudaStream_t st);

namespace {

__global__ void zero_kernel(float* p, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = 0.f;
}

// fill branch: the cache after the step IS X, so dX = g on its S rows.
__global__ void bwd_fill_kernel(BwdStep p) {
    const int u = blockIdx.y;
    const int64_t total = (int64_t)p.S * p.d;
    for (int64_t x = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; x < total; x += (int64_t)gridDim.x * blockDim.x) {
        p.dXK[(int64_t)u * p.S * p.d + x] = p.gK[(int64_t)u * p.M * p.d + x];
        p.dXV[(int64_t)u * p.S * p.d + x] = p.gV[(int64_t)u * p.M * p.d + x];
    }
}

// dw[u][i][j] = <gK[u][i], XK[j]> + <gV[u][i], XV[j]>.  64 slots x 64 positions per block.
template <typename T>
__global__ void __launch_bounds__(256) bwd_dw_kernel(BwdStep p) {
    __shared__ float Gs[64][33];
    __shared__ float Xs[64][33];
    const int u = blockIdx.z, n = u / p.heads, h = u % p.heads;
    const int j0 = blockIdx.x * 64, i0 = blockIdx.y * 64;
    const int tid = threadIdx.x, tj = tid % 16, ti = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
    for (int ch0 = 0; ch0 < 2 * p.d; ch0 += 32) {
        const bool is_v = ch0 >= p.d;
        const int c0 = is_v ? ch0 - p.d : ch0;
        const float* g = (is_v ? p.gV : p.gK) + (int64_t)u * p.M * p.d;
        __syncthreads();
        for (int x = tid; x < 64 * 32; x += 256) {
            const int r = x / 32, cc = x % 32;
            Gs[r][cc] = (i0 + r < p.M) ? g[(int64_t)(i0 + r) * p.d + c0 + cc] : 0.f;
            const int j = j0 + r;
            Xs[r][cc] = (j < p.S) ? to_f32(cat_row<T>(is_v ? p.xv : p.xk, n, h, j)[c0 + cc]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int cc = 0; cc < 32; ++cc) {
            float a[4], z[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) a[x] = Gs[ti + 16 * x][cc];
#pragma unroll
            for (int y = 0; y < 4; ++y) z[y] = Xs[tj + 16 * y][cc];
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], z[y], acc[x][y]);
        }
    }
    float* out = p.dA + (int64_t)u * p.M * p.S;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int i = i0 + ti + 16 * x;
        if (i >= p.M) continue;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int j = j0 + tj + 16 * y;
            if (j < p.S) out[(int64_t)i * p.S + j] = acc[x][y];
        }
    }
}

// One warp per (unit, slot) row: inner = <dw, R>/s;  dA = [R>0] (dw - inner)/s;  dbias += sum_j dA.
__global__ void bwd_dA_kernel(BwdStep p) {
    const int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    if (row >= p.units * p.M) return;
    const int lane = threadIdx.x % 32;
    const int u = row / p.M, i = row % p.M, h = u % p.heads;
    const float* R = p.R + (int64_t)row * p.S;
    float* dA = p.dA + (int64_t)row * p.S;
    const float inv_s = 1.f / p.s[row];
    float inner = 0.f;
    for (int j = lane; j < p.S; j += 32) inner = fmaf(dA[j], R[j], inner);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) inner += __shfl_xor_sync(0xffffffffu, inner, o);
    inner *= inv_s;
    float bsum = 0.f;
    for (int j = lane; j < p.S; j += 32) {
        const float v = R[j] > 0.f ? (dA[j] - inner) * inv_s : 0.f;
        dA[j] = v;
        bsum += v;
    }
    if (p.dbias) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bsum += __shfl_xor_sync(0xffffffffu, bsum, o);
        if (lane == 0) atomicAdd(p.dbias + (p.weights_per_head ? h * p.M : 0) + i, bsum);
    }
}

// dXK[j][:] += sum_i (R[i][j]/s_i) gK[i][:], dXV likewise: the blend's own input gradient.
// Block: POS positions x D channels; 256 threads, 4 positions x 4 channels each.
template <int D>
__global__ void __launch_bounds__(256) bwd_dx_blend_kernel(BwdStep p) {
    constexpr int TX = D / 4, TY = 256 / TX, POS = TY * 4, IT = 32;
    __shared__ float Ws[IT][POS + 1];
    __shared__ __align__(16) float Ks[IT][D];
    __shared__ __align__(16) float Vs[IT][D];
    const int u = blockIdx.y, j0 = blockIdx.x * POS;
    const int tid = threadIdx.x, tx = tid % TX, ty = tid / TX;
    float aK[4][4], aV[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) aK[x][y] = aV[x][y] = 0.f;
    for (int i0 = 0; i0 < p.M; i0 += IT) {
        __syncthreads();
        for (int x = tid; x < IT * POS; x += 256) {
            const int r = x / POS, jj = x % POS;
            const int i = i0 + r, j = j0 + jj;
            Ws[r][jj] = (i < p.M && j < p.S) ? p.R[((int64_t)u * p.M + i) * p.S + j] / p.s[(int64_t)u * p.M + i] : 0.f;
        }
        for (int x = tid; x < IT * D; x += 256) {
            const int r = x / D, ch = x % D;
            const int i = i0 + r;
            Ks[r][ch] = i < p.M ? p.gK[((int64_t)u * p.M + i) * D + ch] : 0.f;
            Vs[r][ch] = i < p.M ? p.gV[((int64_t)u * p.M + i) * D + ch] : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int r = 0; r < IT; ++r) {
            const float4 kx = *reinterpret_cast<const float4*>(&Ks[r][tx * 4]);
            const float4 vx = *reinterpret_cast<const float4*>(&Vs[r][tx * 4]);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float w = Ws[r][ty * 4 + x];
                aK[x][0] = fmaf(w, kx.x, aK[x][0]); aK[x][1] = fmaf(w, kx.y, aK[x][1]);
                aK[x][2] = fmaf(w, kx.z, aK[x][2]); aK[x][3] = fmaf(w, kx.w, aK[x][3]);
                aV[x][0] = fmaf(w, vx.x, aV[x][0]); aV[x][1] = fmaf(w, vx.y, aV[x][1]);
                aV[x][2] = fmaf(w, vx.z, aV[x][2]); aV[x][3] = fmaf(w, vx.w, aV[x][3]);
            }
        }
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int j = j0 + ty * 4 + x;
        if (j >= p.S) continue;
        float* dk = p.dXK + ((int64_t)u * p.S + j) * D + tx * 4;
        float* dv = p.dXV + ((int64_t)u * p.S + j) * D + tx * 4;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            dk[y] += aK[x][y];
            dv[y] += aV[x][y];
        }
    }
}

// Conv input Z[j][ch] of unit (n,h): keys for ch < d, values for ch >= d.
template <typename T>
__device__ __forceinline__ float conv_input(const BwdStep& p, int n, int h, int j, int ch) {
    if (j < 0 || j >= p.S) return 0.f;
    return ch < p.d ? to_f32(cat_row<T>(p.xk, n, h, j)[ch]) : to_f32(cat_row<T>(p.xv, n, h, j)[ch - p.d]);
}

// dG[set][i][ch][t] += sum over the set's units, sum_j dA[u][i][j] * Z_u[j+t-pad][ch].
// Block: 32 slots x 32 channels, taps in groups of 8, a few units of one weight set per block
// (their contributions are summed in registers; blocks of the same set combine by atomicAdd).
constexpr int GT = 8;    // taps per pass
constexpr int GJ = 64;   // positions per stage
template <typename T>
__global__ void __launch_bounds__(256) bwd_dG_kernel(BwdStep p, int units_per_block, int groups) {
    __shared__ float As[32][GJ + 1];
    __shared__ float Zs[GJ + GT - 1][33];
    const int set = blockIdx.z / groups, group = blockIdx.z % groups;
    const int units_in_set = p.weights_per_head ? p.units / p.heads : p.units;
    const int ch0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
    const int tid = threadIdx.x, cl = tid % 32, ig = tid / 32;
    const int pad = (p.k - 1) / 2;
    for (int t0 = 0; t0 < p.k; t0 += GT) {
        float acc[4][GT];
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int t = 0; t < GT; ++t) acc[x][t] = 0.f;
        for (int m = group * units_per_block; m < min(units_in_set, (group + 1) * units_per_block); ++m) {
            const int u = p.weights_per_head ? m * p.heads + set : m;
            const int n = u / p.heads, h = u % p.heads;
            const float* dA = p.dA + (int64_t)u * p.M * p.S;
            for (int j0 = 0; j0 < p.S; j0 += GJ) {
                __syncthreads();
                for (int x = tid; x < 32 * GJ; x += 256) {
                    const int r = x / GJ, jj = x % GJ;
                    As[r][jj] = (i0 + r < p.M && j0 + jj < p.S) ? dA[(int64_t)(i0 + r) * p.S + j0 + jj] : 0.f;
                }
                for (int x = tid; x < (GJ + GT - 1) * 32; x += 256) {
                    const int r = x / 32, cc = x % 32;
                    Zs[r][cc] = (ch0 + cc < p.c_in) ? conv_input<T>(p, n, h, j0 + r + t0 - pad, ch0 + cc) : 0.f;
                }
                __syncthreads();
#pragma unroll 4
                for (int jj = 0; jj < GJ; ++jj) {
                    float a[4], z[GT];
#pragma unroll
                    for (int x = 0; x < 4; ++x) a[x] = As[ig * 4 + x][jj];
#pragma unroll
                    for (int t = 0; t < GT; ++t) z[t] = Zs[jj + t][cl];
#pragma unroll
                    for (int x = 0; x < 4; ++x)
#pragma unroll
                        for (int t = 0; t < GT; ++t) acc[x][t] = fmaf(a[x], z[t], acc[x][t]);
                }
            }
        }
        const int ch = ch0 + cl;
        if (ch < p.c_in) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int i = i0 + ig * 4 + x;
                if (i >= p.M) continue;
                float* out = p.dG + (((int64_t)set * p.M + i) * p.c_in + ch) * p.k;
#pragma unroll
                for (int t = 0; t < GT; ++t)
                    if (t0 + t < p.k) atomicAdd(out + t0 + t, acc[x][t]);
            }
        }
    }
}

// dZ[j'][ch] = sum_i sum_t dA[i][j'-t+pad] * G[i][ch][t], added into dXK (ch < d) or dXV (ch >= d).
// Block: 64 positions x 64 channels, 4x4 outputs per thread (strided by 16).
template <typename T>
__global__ void __launch_bounds__(256) bwd_dZ_kernel(BwdStep p) {
    extern __shared__ float smem[];
    const int acols = 64 + p.k - 1;
    float* As = smem;                     // [32 slots][acols + 1]
    float* Gs = smem + 32 * (acols + 1);  // [32 slots][65]
    const int u = blockIdx.z, h = u % p.heads;
    const int j0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
    const int tid = threadIdx.x, tj = tid % 16, tc = tid / 16;
    const int pad = (p.k - 1) / 2;
    const T* gp = reinterpret_cast<const T*>(p.g_packed) + (p.weights_per_head ? (int64_t)h * p.k * p.M * p.c_in : 0);
    const float* dA = p.dA + (int64_t)u * p.M * p.S;
    float acc[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
    for (int i0 = 0; i0 < p.M; i0 += 32) {
        __syncthreads();
        for (int x = tid; x < 32 * acols; x += 256) {
            const int r = x / acols, cc = x % acols;
            const int j = j0 - pad + cc;
            As[r * (acols + 1) + cc] = (i0 + r < p.M && j >= 0 && j < p.S) ? dA[(int64_t)(i0 + r) * p.S + j] : 0.f;
        }
        for (int t = 0; t < p.k; ++t) {
            __syncthreads();
            for (int x = tid; x < 32 * 64; x += 256) {
                const int r = x / 64, cc = x % 64;
                Gs[r * 65 + cc] = (i0 + r < p.M && c0 + cc < p.c_in)
                                      ? to_f32(gp[((int64_t)t * p.M + i0 + r) * p.c_in + c0 + cc]) : 0.f;
            }
            __syncthreads();
            const int off = p.k - 1 - t;  // column of dA[., j'-t+pad] in the staged window
#pragma unroll 8
            for (int r = 0; r < 32; ++r) {
                float a[4], g[4];
#pragma unroll
                for (int y = 0; y < 4; ++y) a[y] = As[r * (acols + 1) + tj + 16 * y + off];
#pragma unroll
                for (int x = 0; x < 4; ++x) g[x] = Gs[r * 65 + tc + 16 * x];
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(g[x], a[y], acc[x][y]);
            }
        }
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int ch = c0 + tc + 16 * x;
        if (ch >= p.c_in) continue;
        float* dst = (ch < p.d ? p.dXK : p.dXV) + (int64_t)u * p.S * p.d + (ch < p.d ? ch : ch - p.d);
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int j = j0 + tj + 16 * y;
            if (j < p.S) dst[(int64_t)j * p.d] += acc[x][y];
        }
    }
}

// delta[u][r] = <dO_r, O_r>: one warp per query row.
template <typename T>
__global__ void bwd_delta_kernel(BwdStep p) {
    const int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    if (row >= p.units * p.b) return;
    const int lane = threadIdx.x % 32, u = row / p.b, r = row % p.b, n = u / p.heads, h = u % p.heads;
    const T* o = unit_base<T>(p.o, n, h) + (int64_t)r * p.o.st;
    const T* g = unit_base<T>(p.d_o, n, h) + (int64_t)r * p.d_o.st;
    float acc = 0.f;
    for (int ch = lane; ch < p.d; ch += 32) acc = fmaf(to_f32(o[ch]), to_f32(g[ch]), acc);
#pragma unroll
    for (int of = 16; of > 0; of >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, of);
    if (lane == 0) p.delta[row] = acc;
}

__device__ __forceinline__ float quad_sum(float x) {
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    return x;
}
__device__ __forceinline__ float dot4(const float4& a, const float4& b, float acc) {
    acc = fmaf(a.x, b.x, acc); acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc); acc = fmaf(a.w, b.w, acc);
    return acc;
}
__device__ __forceinline__ void axpy4(float s, const float4& x, float4& y) {
    y.x = fmaf(s, x.x, y.x); y.y = fmaf(s, x.y, y.y); y.z = fmaf(s, x.z, y.z); y.w = fmaf(s, x.w, y.w);
}

// dQ of Eq. 1: 32 queries per block, 4 threads per query (interleaved float4 channel groups).
template <typename T, int D>
__global__ void __launch_bounds__(128) bwd_attn_dq_kernel(BwdStep p) {
    constexpr int NV = D / 16, KT = 32;
    __shared__ __align__(16) float Ks[KT][D];
    __shared__ __align__(16) float Vs[KT][D];
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int tid = threadIdx.x, m = tid % 4;
    const int r = blockIdx.x * 32 + tid / 4;
    const bool live = r < p.b;
    const int rr = live ? r : 0;
    const float sc2 = p.scale * 1.4426950408889634f;
    float4 q[NV], g[NV], dq[NV];
    const T* qrow = unit_base<T>(p.q, n, h) + (int64_t)rr * p.q.st;
    const T* grow = unit_base<T>(p.d_o, n, h) + (int64_t)rr * p.d_o.st;
#pragma unroll
    for (int e = 0; e < NV; ++e) {
        const int ch = 4 * (m + 4 * e);
        q[e] = make_float4(to_f32(qrow[ch]), to_f32(qrow[ch + 1]), to_f32(qrow[ch + 2]), to_f32(qrow[ch + 3]));
        g[e] = make_float4(to_f32(grow[ch]), to_f32(grow[ch + 1]), to_f32(grow[ch + 2]), to_f32(grow[ch + 3]));
        dq[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const float lse2 = p.lse[(int64_t)u * p.lse_stride + rr] * 1.4426950408889634f;
    const float delta = p.delta[(int64_t)u * p.b + rr];
    const int last_row = min((int)blockIdx.x * 32 + 31, p.b - 1);
    const int ncols = p.c + last_row + 1, my_cols = p.c + r + 1;
    for (int j0 = 0; j0 < ncols; j0 += KT) {
        __syncthreads();
        for (int x = tid; x < KT * D; x += 128) {
            const int jj = x / D, ch = x % D, j = j0 + jj;
            Ks[jj][ch] = j < p.S ? to_f32(cat_row<T>(p.xk, n, h, j)[ch]) : 0.f;
            Vs[jj][ch] = j < p.S ? to_f32(cat_row<T>(p.xv, n, h, j)[ch]) : 0.f;
        }
        __syncthreads();
#pragma unroll 2
        for (int jj = 0; jj < KT; ++jj) {
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int e = 0; e < NV; ++e) {
                s = dot4(q[e], *reinterpret_cast<const float4*>(&Ks[jj][4 * (m + 4 * e)]), s);
                dp = dot4(g[e], *reinterpret_cast<const float4*>(&Vs[jj][4 * (m + 4 * e)]), dp);
            }
            s = quad_sum(s);
            dp = quad_sum(dp);
            const float pr = (live && j0 + jj < my_cols) ? exp2f(s * sc2 - lse2) : 0.f;
            const float ds = pr * (dp - delta) * p.scale;
#pragma unroll
            for (int e = 0; e < NV; ++e) axpy4(ds, *reinterpret_cast<const float4*>(&Ks[jj][4 * (m + 4 * e)]), dq[e]);
        }
    }
    if (!live) return;
    T* out = unit_base_mut<T>(p.dq, n, h) + (int64_t)r * p.dq.st;
#pragma unroll
    for (int e = 0; e < NV; ++e) {
        const int ch = 4 * (m + 4 * e);
        out[ch] = from_f32<T>(dq[e].x); out[ch + 1] = from_f32<T>(dq[e].y);
        out[ch + 2] = from_f32<T>(dq[e].z); out[ch + 3] = from_f32<T>(dq[e].w);
    }
}

// dK, dV of Eq. 1 added into dXK, dXV: 32 keys of [cache; chunk] per block, 4 threads per key.
template <typename T, int D>
__global__ void __launch_bounds__(128) bwd_attn_dkv_kernel(BwdStep p) {
    constexpr int NV = D / 16, QT = 32;
    __shared__ __align__(16) float Qs[QT][D];
    __shared__ __align__(16) float Gs[QT][D];
    __shared__ float lse_s[QT], delta_s[QT];
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int tid = threadIdx.x, m = tid % 4;
    const int j = blockIdx.x * 32 + tid / 4;
    const bool live = j < p.S;
    const int jr = live ? j : 0;
    const float sc2 = p.scale * 1.4426950408889634f;
    float4 kk[NV], vv[NV], dk[NV], dv[NV];
    const T* krow = cat_row<T>(p.xk, n, h, jr);
    const T* vrow = cat_row<T>(p.xv, n, h, jr);
#pragma unroll
    for (int e = 0; e < NV; ++e) {
        const int ch = 4 * (m + 4 * e);
        kk[e] = make_float4(to_f32(krow[ch]), to_f32(krow[ch + 1]), to_f32(krow[ch + 2]), to_f32(krow[ch + 3]));
        vv[e] = make_float4(to_f32(vrow[ch]), to_f32(vrow[ch + 1]), to_f32(vrow[ch + 2]), to_f32(vrow[ch + 3]));
        dk[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        dv[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // key j is visible to query r iff j <= c + r; the block's first key bounds the first query tile
    const int r_first = max(0, (int)blockIdx.x * 32 - p.c);
    for (int r0 = (r_first / QT) * QT; r0 < p.b; r0 += QT) {
        __syncthreads();
        for (int x = tid; x < QT * D; x += 128) {
            const int rr = x / D, ch = x % D, r = r0 + rr;
            Qs[rr][ch] = r < p.b ? to_f32((unit_base<T>(p.q, n, h) + (int64_t)r * p.q.st)[ch]) : 0.f;
            Gs[rr][ch] = r < p.b ? to_f32((unit_base<T>(p.d_o, n, h) + (int64_t)r * p.d_o.st)[ch]) : 0.f;
        }
        if (tid < QT) {
            const int r = r0 + tid;
            lse_s[tid] = r < p.b ? p.lse[(int64_t)u * p.lse_stride + r] * 1.4426950408889634f : 0.f;
            delta_s[tid] = r < p.b ? p.delta[(int64_t)u * p.b + r] : 0.f;
        }
        __syncthreads();
#pragma unroll 2
        for (int rr = 0; rr < QT; ++rr) {
            const int r = r0 + rr;
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int e = 0; e < NV; ++e) {
                s = dot4(kk[e], *reinterpret_cast<const float4*>(&Qs[rr][4 * (m + 4 * e)]), s);
                dp = dot4(vv[e], *reinterpret_cast<const float4*>(&Gs[rr][4 * (m + 4 * e)]), dp);
            }
            s = quad_sum(s);
            dp = quad_sum(dp);
            const float pr = (live && r < p.b && j <= p.c + r) ? exp2f(s * sc2 - lse_s[rr]) : 0.f;
            const float ds = pr * (dp - delta_s[rr]) * p.scale;
#pragma unroll
            for (int e = 0; e < NV; ++e) {
                axpy4(ds, *reinterpret_cast<const float4*>(&Qs[rr][4 * (m + 4 * e)]), dk[e]);
                axpy4(pr, *reinterpret_cast<const float4*>(&Gs[rr][4 * (m + 4 * e)]), dv[e]);
            }
        }
    }
    if (!live) return;
    float* ok = p.dXK + ((int64_t)u * p.S + j) * D;
    float* ov = p.dXV + ((int64_t)u * p.S + j) * D;
#pragma unroll
    for (int e = 0; e < NV; ++e) {
        const int ch = 4 * (m + 4 * e);
        ok[ch] += dk[e].x; ok[ch + 1] += dk[e].y; ok[ch + 2] += dk[e].z; ok[ch + 3] += dk[e].w;
        ov[ch] += dv[e].x; ov[ch + 1] += dv[e].y; ov[ch + 2] += dv[e].z; ov[ch + 3] += dv[e].w;
    }
}

// Rows 0..c-1 of dX become the gradient w.r.t. the cache before this step (rows >= c: zero);
// rows c..S-1 are this chunk's dK, dV.
template <typename T>
__global__ void bwd_split_kernel(BwdStep p) {
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int rows = max(p.M, p.S);
    const int64_t total = (int64_t)rows * p.d;
    for (int64_t x = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; x < total; x += (int64_t)gridDim.x * blockDim.x) {
        const int row = x / p.d, ch = x % p.d;
        const float dk = row < p.S ? p.dXK[((int64_t)u * p.S + row) * p.d + ch] : 0.f;
        const float dv = row < p.S ? p.dXV[((int64_t)u * p.S + row) * p.d + ch] : 0.f;
        if (row < p.M) {
            p.gK[((int64_t)u * p.M + row) * p.d + ch] = row < p.c ? dk : 0.f;
            p.gV[((int64_t)u * p.M + row) * p.d + ch] = row < p.c ? dv : 0.f;
        }
        if (row >= p.c && row < p.S) {
            unit_base_mut<T>(p.dk, n, h)[(int64_t)(row - p.c) * p.dk.st + ch] = from_f32<T>(dk);
            unit_base_mut<T>(p.dv, n, h)[(int64_t)(row - p.c) * p.dv.st + ch] = from_f32<T>(dv);
        }
    }
}

// g = gradient of the loss w.r.t. the final cache (zero where the caller passes none).
template <typename T>
__global__ void bwd_init_g_kernel(View gk_in, View gv_in, float* gK, float* gV, int heads, int M, int d) {
    const int u = blockIdx.y, n = u / heads, h = u % heads;
    const int total = M * d;
    for (int x = blockIdx.x * blockDim.x + threadIdx.x; x < total; x += gridDim.x * blockDim.x) {
        const int row = x / d, ch = x % d;
        gK[(int64_t)u * total + x] = gk_in.ptr ? to_f32((unit_base<T>(gk_in, n, h) + (int64_t)row * gk_in.st)[ch]) : 0.f;
        gV[(int64_t)u * total + x] = gv_in.ptr ? to_f32((unit_base<T>(gv_in, n, h) + (int64_t)row * gv_in.st)[ch]) : 0.f;
    }
}

// The gradient w.r.t. the cache the loop started from, out of the fp32 accumulators (all M rows; rows beyond the
// initial fill count hold zeros).
template <typename T>
__global__ void bwd_store_g_kernel(const float* gK, const float* gV, View gk_out, View gv_out, int heads, int M, int d) {
    const int u = blockIdx.y, n = u / heads, h = u % heads;
    const int total = M * d;
    for (int x = blockIdx.x * blockDim.x + threadIdx.x; x < total; x += gridDim.x * blockDim.x) {
        const int row = x / d, ch = x % d;
        if (gk_out.ptr) unit_base_mut<T>(gk_out, n, h)[(int64_t)row * gk_out.st + ch] = from_f32<T>(gK[(int64_t)u * total + x]);
        if (gv_out.ptr) unit_base_mut<T>(gv_out, n, h)[(int64_t)row * gv_out.st + ch] = from_f32<T>(gV[(int64_t)u * total + x]);
    }
}

bool launched() { return cudaGetLastError() == cudaSuccess; }

// All kernels of one reversed step. Returns the number of launches or -1.
// `tb` (tensor-core scratch) non-null: the contractions run as tcgen05 GEMMs (tensor_backward.cu).
template <typename T>
int backward_step(lococo_handle* h, const BwdStep& p, const CompressParams& fwd, int dtype, int B, char* tb, cudaStream_t st) {
    int n = 0;
    if (tb) {
        const int r = tensor_backward_pack(h, p, B, tb, st);
        if (r < 0) return -1;
        n += r;
    }
    const int64_t dx = (int64_t)p.units * p.S * p.d;
    const int zb = (int)std::min<int64_t>((dx + 255) / 256, 4096);
    if (p.c + p.b <= p.M) {
        bwd_fill_kernel<<<dim3(std::min<int64_t>(((int64_t)p.S * p.d + 255) / 256, 1024), p.units), 256, 0, st>>>(p);
        if (!launched()) return -1;
        ++n;
    } else {
        zero_kernel<<<zb, 256, 0, st>>>(p.dXK, dx);
        zero_kernel<<<zb, 256, 0, st>>>(p.dXV, dx);
        if (!launched()) return -1;
        n += 2;
        if (tb) {
            const int r = tensor_backward_compress(h, p, fwd, B, tb, st);
            if (r < 0) return -1;
            n += r;
        } else {
        const int r = simt_conv_rowsum(dtype, fwd, st);   // R and s of the forward, recomputed
        if (r < 0) return -1;
        n += r;
        bwd_dw_kernel<T><<<dim3((p.S + 63) / 64, (p.M + 63) / 64, p.units), 256, 0, st>>>(p);
        bwd_dA_kernel<<<(p.units * p.M + 7) / 8, 256, 0, st>>>(p);
        if (p.d == 128) bwd_dx_blend_kernel<128><<<dim3((p.S + 31) / 32, p.units), 256, 0, st>>>(p);
        else bwd_dx_blend_kernel<64><<<dim3((p.S + 63) / 64, p.units), 256, 0, st>>>(p);
        if (!launched()) return -1;
        n += 3;
        const int sets = p.weights_per_head ? p.heads : 1;
        const int in_set = p.units / sets;
        const int upb = in_set >= 4 ? 4 : in_set;
        const int groups = (in_set + upb - 1) / upb;
        bwd_dG_kernel<T><<<dim3((p.c_in + 31) / 32, (p.M + 31) / 32, sets * groups), 256, 0, st>>>(p, upb, groups);
        const size_t smem = sizeof(float) * (32 * (64 + p.k) + 32 * 65);
        bwd_dZ_kernel<T><<<dim3((p.S + 63) / 64, (p.c_in + 63) / 64, p.units), 256, smem, st>>>(p);
        if (!launched()) return -1;
        n += 2;
        }
    }
    bwd_delta_kernel<T><<<(p.units * p.b + 7) / 8, 256, 0, st>>>(p);
    if (tb) {
        if (!launched()) return -1;
        const int r = tensor_backward_attention(h, p, B, tb, st);
        if (r < 0) return -1;
        n += r - 2;
    } else if (p.d == 128) {
        bwd_attn_dq_kernel<T, 128><<<dim3((p.b + 31) / 32, p.units), 128, 0, st>>>(p);
        bwd_attn_dkv_kernel<T, 128><<<dim3((p.S + 31) / 32, p.units), 128, 0, st>>>(p);
    } else {
        bwd_attn_dq_kernel<T, 64><<<dim3((p.b + 31) / 32, p.units), 128, 0, st>>>(p);
        bwd_attn_dkv_kernel<T, 64><<<dim3((p.S + 31) / 32, p.units), 128, 0, st>>>(p);
    }
    const int rows = std::max(p.M, p.S);
    bwd_split_kernel<T><<<dim3(std::min<int64_t>(((int64_t)rows * p.d + 255) / 256, 1024), p.units), 256, 0, st>>>(p);
    if (!launched()) return -1;
    return n + 4;
}

template <typename T>
int init_g(View gk, View gv, float* gK, float* gV, int heads, int units, int M, int d, cudaStream_t st) {
    bwd_init_g_kernel<T><<<dim3((M * d + 255) / 256, units), 256, 0, st>>>(gk, gv, gK, gV, heads, M, d);
    return launched() ? 1 : -1;
}

template <typename T>
int store_g(const float* gK, const float* gV, View gk, View gv, int heads, int units, int M, int d, cudaStream_t st) {
    bwd_store_g_kernel<T><<<dim3((M * d + 255) / 256, units), 256, 0, st>>>(gK, gV, gk, gv, heads, M, d);
    return launched() ? 1 : -1;
}

}  // namespace
}  // namespace lococo

using namespace lococo;

namespace {

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

bool bview_ok(const lococo_tensor& t, size_t elt) {
    if (!t.ptr || (reinterpret_cast<uintptr_t>(t.ptr) & 15u)) return false;
    if ((t.stride_batch * (int64_t)elt) % 16 || (t.stride_head * (int64_t)elt) % 16 || (t.stride_token * (int64_t)elt) % 16)
        return false;
    return t.stride_token > 0;
}

View bdev(const lococo_tensor& t, int64_t tokens, size_t elt) {
    View v{static_cast<char*>(t.ptr), t.stride_batch, t.stride_head, t.stride_token};
    if (v.ptr) v.ptr += tokens * t.stride_token * (int64_t)elt;
    return v;
}

struct Scratch {
    size_t gK, gV, dXK, dXV, dA, delta, tensor, total;
};

Scratch scratch_layout(const lococo_handle* h, int B) {
    const lococo_config& c = h->cfg;
    const size_t units = h->units, Smax = (size_t)c.M + B;
    Scratch s{};
    size_t off = 0;
    s.gK = off;    off = align256(off + units * c.M * c.head_dim * sizeof(float));
    s.gV = off;    off = align256(off + units * c.M * c.head_dim * sizeof(float));
    s.dXK = off;   off = align256(off + units * Smax * c.head_dim * sizeof(float));
    s.dXV = off;   off = align256(off + units * Smax * c.head_dim * sizeof(float));
    s.dA = off;    off = align256(off + units * c.M * Smax * sizeof(float));
    s.delta = off; off = align256(off + units * (size_t)B * sizeof(float));
    s.tensor = off;
    if (tensor_backward_supported(h)) off = align256(off + tensor_backward_scratch_bytes(h, B));
    s.total = off;
    return s;
}

}  // namespace

extern "C" {

lococo_status lococo_backward_scratch_bytes(const lococo_handle* h, int32_t L, int32_t B, size_t* out) {
    if (!h || !out || L < 1 || B < 1 || B > h->cfg.max_chunk) return LOCOCO_ERR_INVALID_ARG;
    *out = scratch_layout(h, B).total;
    return LOCOCO_OK;
}

lococo_status lococo_process_sequence_backward(lococo_handle* h, lococo_tensor Q, lococo_tensor K, lococo_tensor V,
                                               lococo_tensor O, int32_t L, int32_t B, int32_t cache_len_in, const void* saved,
                                               lococo_tensor dO, lococo_tensor dKc_final, lococo_tensor dVc_final,
                                               lococo_tensor dQ, lococo_tensor dK, lococo_tensor dV, float* dG, float* dbias,
                                               lococo_tensor dKc_in, lococo_tensor dVc_in, void* scratch,
                                               size_t scratch_bytes, void* stream) {
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    if (!h->ws || !h->weights_set) return LOCOCO_ERR_WORKSPACE;
    const lococo_config& cfg = h->cfg;
    if (L < 1 || B < 1 || B > cfg.max_chunk || !saved || !dG || !scratch) return LOCOCO_ERR_INVALID_ARG;
    if (cache_len_in < 0 || cache_len_in > cfg.M) return LOCOCO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(saved) & 255u) || (reinterpret_cast<uintptr_t>(scratch) & 255u) ||
        (reinterpret_cast<uintptr_t>(dG) & 15u))
        return LOCOCO_ERR_INVALID_ARG;
    const size_t e = h->elt;
    if (!bview_ok(Q, e) || !bview_ok(K, e) || !bview_ok(V, e) || !bview_ok(O, e) || !bview_ok(dO, e) || !bview_ok(dQ, e) ||
        !bview_ok(dK, e) || !bview_ok(dV, e))
        return LOCOCO_ERR_INVALID_ARG;
    if ((dKc_final.ptr && !bview_ok(dKc_final, e)) || (dVc_final.ptr && !bview_ok(dVc_final, e))) return LOCOCO_ERR_INVALID_ARG;
    if ((dKc_in.ptr && !bview_ok(dKc_in, e)) || (dVc_in.ptr && !bview_ok(dVc_in, e))) return LOCOCO_ERR_INVALID_ARG;
    if (dbias && !h->has_bias) return LOCOCO_ERR_INVALID_ARG;
    const Scratch sl = scratch_layout(h, B);
    if (scratch_bytes < sl.total) return LOCOCO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* sc = static_cast<char*>(scratch);
    float* gK = reinterpret_cast<float*>(sc + sl.gK);
    float* gV = reinterpret_cast<float*>(sc + sl.gV);

    const int n_chunks = (L + B - 1) / B;
    const size_t snap_step = (size_t)h->units * cfg.M * cfg.head_dim * e;
    const size_t snap_all = align256((size_t)n_chunks * snap_step);
    const char* sv = static_cast<const char*>(saved);
    const float* lse_all = reinterpret_cast<const float*>(sv + 2 * snap_all);

    char* tb = tensor_backward_supported(h) ? sc + sl.tensor : nullptr;
    if (tb) {
        const int r = tensor_backward_prepare(h, B, tb, st);
        if (r < 0) return LOCOCO_ERR_CUDA;
        h->launches += r;
    }
    int launched_n = cfg.dtype == LOCOCO_F32
                         ? init_g<float>(bdev(dKc_final, 0, e), bdev(dVc_final, 0, e), gK, gV, cfg.heads, h->units, cfg.M, cfg.head_dim, st)
                         : init_g<__nv_bfloat16>(bdev(dKc_final, 0, e), bdev(dVc_final, 0, e), gK, gV, cfg.heads, h->units, cfg.M,
                                                 cfg.head_dim, st);
    if (launched_n < 0) return LOCOCO_ERR_CUDA;
    h->launches += launched_n;

    // cache fill count before every step of the forward
    int c_before[4096];
    if (n_chunks > 4096) return LOCOCO_ERR_UNSUPPORTED_SHAPE;
    for (int n = 0, c = cache_len_in; n < n_chunks; ++n) {
        const int b = std::min(B, L - n * B);
        c_before[n] = c;
        c = c + b <= cfg.M ? c + b : cfg.M;
    }
    for (int n = n_chunks - 1; n >= 0; --n) {
        const int t0 = n * B, b = std::min(B, L - t0), c = c_before[n];
        lococo_tensor snapK{const_cast<char*>(sv) + (size_t)n * snap_step, (int64_t)cfg.heads * cfg.M * cfg.head_dim,
                            (int64_t)cfg.M * cfg.head_dim, (int64_t)cfg.head_dim};
        lococo_tensor snapV = snapK;
        snapV.ptr = const_cast<char*>(sv) + snap_all + (size_t)n * snap_step;
        BwdStep p{};
        p.xk = CatView{bdev(snapK, 0, e), bdev(K, t0, e), c, b};
        p.xv = CatView{bdev(snapV, 0, e), bdev(V, t0, e), c, b};
        p.q = bdev(Q, t0, e); p.o = bdev(O, t0, e); p.d_o = bdev(dO, t0, e);
        p.dq = bdev(dQ, t0, e); p.dk = bdev(dK, t0, e); p.dv = bdev(dV, t0, e);
        p.heads = cfg.heads; p.units = h->units; p.d = cfg.head_dim; p.M = cfg.M; p.k = cfg.k; p.c_in = cfg.c_in;
        p.c = c; p.b = b; p.S = c + b;
        p.weights_per_head = cfg.weights_per_head;
        p.g_packed = h->ws + h->off_gpack;
        p.scale = h->scale;
        p.lse = lse_all + t0; p.lse_stride = L;
        p.R = reinterpret_cast<float*>(h->ws + h->off_R);
        p.s = reinterpret_cast<float*>(h->ws + h->off_s);
        p.dA = reinterpret_cast<float*>(sc + sl.dA);
        p.delta = reinterpret_cast<float*>(sc + sl.delta);
        p.gK = gK; p.gV = gV;
        p.dXK = reinterpret_cast<float*>(sc + sl.dXK);
        p.dXV = reinterpret_cast<float*>(sc + sl.dXV);
        p.dG = dG; p.dbias = dbias;
        CompressParams f{};
        f.xk = p.xk; f.xv = p.xv;
        f.heads = cfg.heads; f.units = h->units; f.d = cfg.head_dim; f.M = cfg.M; f.k = cfg.k; f.c_in = cfg.c_in;
        f.S = p.S; f.weights_per_head = cfg.weights_per_head; f.g_packed = p.g_packed;
        f.bias = h->has_bias ? reinterpret_cast<const float*>(h->ws + h->off_bias) : nullptr;
        f.eps = cfg.norm_eps; f.prot = h->prot; f.R = p.R; f.s = p.s;
        const int r = cfg.dtype == LOCOCO_F32 ? backward_step<float>(h, p, f, cfg.dtype, B, nullptr, st)
                                              : backward_step<__nv_bfloat16>(h, p, f, cfg.dtype, B, tb, st);
        if (r < 0) return LOCOCO_ERR_CUDA;
        h->launches += r;
    }
    // what the accumulators hold now is the gradient w.r.t. the cache the forward started from
    if (dKc_in.ptr || dVc_in.ptr) {
        const int r = cfg.dtype == LOCOCO_F32
                          ? store_g<float>(gK, gV, bdev(dKc_in, 0, e), bdev(dVc_in, 0, e), cfg.heads, h->units, cfg.M, cfg.head_dim, st)
                          : store_g<__nv_bfloat16>(gK, gV, bdev(dKc_in, 0, e), bdev(dVc_in, 0, e), cfg.heads, h->units, cfg.M,
                                                   cfg.head_dim, st);
        if (r < 0) return LOCOCO_ERR_CUDA;
        h->launches += r;
    }
    return LOCOCO_OK;
}

}  // extern "C"
