// Backward pass of Algorithm 2 on the tensor cores (bf16 storage, d = 128, M a multiple of 128).
// Every contraction of one reversed step is a launch of the batched GEMM of gemm_tc.cuh on operands
// that small packing kernels lay out once per step:
//   cache update (Eq. 4-7 reversed)
//     R, s        recomputed by the forward's own tcgen05 conv kernel (R left in place)
//     dw          = [gK | gV] [X_K | X_V]^T                          per unit, K = 2d
//     dA          row kernel: dA = [R>0] (dw - <dw, w>_row) / s with w = R / s, rounded to bf16
//     dX         += w^T [gK | gV] = R^T ([gK | gV] / s)               per unit, K = M; R is exact in bf16
//     dG         += sum over units and positions of dA (*) Z          the im2col view of Z is a tensor
//                                                                     map with overlapping strides
//     dZ (in dX) += sum over taps of shift_t(dA^T) G_t                a tap = a row offset of the box
//   attention (Eq. 1 reversed), in blocks of up to 1024 queries, P and dS materialised in bf16:
//     P = exp(scale Q X_K^T - lse), dS = scale P (dO X_V^T - delta)   one launch, two accumulators per tile, softmax
//                                                                     and its gradient in the epilogue; masked tiles skipped
//     dX_V += P^T dO, dX_K += dS^T Q, dQ = dS X_K                     K loops cut at the causal limit
// Gradients that enter a GEMM are rounded to bf16 (fp32 accumulation), like the forward's operands; the
// cache gradient, which every earlier step inherits, enters as two bf16 terms (value + remainder).
#include <algorithm>

#include "backward.h"
#include "gemm_tc.cuh"
#include "handle.h"

namespace lococo {
namespace {

constexpr int kD = 128;
constexpr int kQBlock = 1024;   // queries per attention block

size_t align256(size_t x) { return (x + 255) / 256 * 256; }
int round_up(int x, int m) { return (x + m - 1) / m * m; }

struct Layout {
    int Sp, Sp2, QB;
    size_t xpad, gkv, gkv_lo, gs, gs_lo, wb, dab, dat, gt, dummy_k, dummy_v, dw, pb, dsb, total;
};

Layout layout_of(const lococo_handle* h, int B) {
    const lococo_config& c = h->cfg;
    const size_t U = h->units, sets = c.weights_per_head ? c.heads : 1;
    Layout L{};
    const int Smax = c.M + B, pad = (c.k - 1) / 2;
    L.Sp = round_up(Smax, 8);
    L.Sp2 = round_up(Smax + 2 * pad, 8);
    L.QB = std::min(round_up(B, 128), kQBlock);
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off = align256(off + bytes); return o; };
    L.xpad = take(U * L.Sp2 * 256 * 2);
    L.gkv = take(U * c.M * 256 * 2);
    L.gkv_lo = take(U * c.M * 256 * 2);
    L.gs = take(U * c.M * 256 * 2);
    L.gs_lo = take(U * c.M * 256 * 2);
    L.wb = take(U * c.M * L.Sp * 2);
    L.dab = take(U * c.M * L.Sp * 2);
    L.dat = take(U * (size_t)L.Sp * c.M * 2);
    L.gt = take(sets * c.k * c.c_in * c.M * 2);
    L.dummy_k = take(U * c.M * kD * 2);
    L.dummy_v = take(U * c.M * kD * 2);
    L.dw = take(U * c.M * L.Sp * 4);
    L.pb = take(U * (size_t)L.QB * L.Sp * 2);
    L.dsb = take(U * (size_t)L.QB * L.Sp * 2);
    L.total = off;
    return L;
}

bool launched() { return cudaGetLastError() == cudaSuccess; }

// ------------------------------------------------------------------ packing kernels
// Xpad[u][pad + j][0:128] = X_K[j], [128:256] = X_V[j]; zero rows above and below (the conv's padding).
__global__ void pack_x_kernel(BwdStep p, __nv_bfloat16* xpad, int Sp2, int pad) {
    const int u = blockIdx.y, n = u / p.heads, h = u % p.heads;
    const int piece = threadIdx.x & 31;                     // 8 channels of the 256-wide row
    for (int jr = blockIdx.x * 8 + (threadIdx.x >> 5); jr < Sp2; jr += gridDim.x * 8) {
        const int j = jr - pad;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (j >= 0 && j < p.S) {
            const CatView& x = piece < 16 ? p.xk : p.xv;
            v = *reinterpret_cast<const uint4*>(cat_row<__nv_bfloat16>(x, n, h, j) + (piece & 15) * 8);
        }
        *reinterpret_cast<uint4*>(xpad + ((int64_t)u * Sp2 + jr) * 256 + piece * 8) = v;
    }
}

// gKV[u][i] = [gK[u][i] | gV[u][i]] in bf16, and the part of it that bf16 drops, also in bf16: dw is
// followed by the subtraction dw - <dw, w> (Eq. 7 reversed), which cancels most of it, so dw is
// computed from both parts (two GEMMs) and carries the gradient to about 16 bits.
// The same split of g / s (row i divided by the denominator s_i of Eq. 7): the blend's own gradient is
// dX = w^T g = R^T (g / s), and R is exact in bf16 (the forward rounded it), so that GEMM loses nothing.
__global__ void pack_g_kernel(const float* gK, const float* gV, const float* s, __nv_bfloat16* gkv, __nv_bfloat16* gkv_lo,
                              __nv_bfloat16* gs, __nv_bfloat16* gs_lo, int64_t rows) {
    const int64_t total = rows * 256;
    for (int64_t x = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; x < total; x += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = x / 256;
        const int ch = (int)(x % 256);
        const float g = ch < kD ? gK[r * kD + ch] : gV[r * kD + ch - kD];
        const __nv_bfloat16 hi = __float2bfloat16_rn(g);
        gkv[x] = hi;
        gkv_lo[x] = __float2bfloat16_rn(g - __bfloat162float(hi));
        const float q = g / s[r];
        const __nv_bfloat16 qh = __float2bfloat16_rn(q);
        gs[x] = qh;
        gs_lo[x] = __float2bfloat16_rn(q - __bfloat162float(qh));
    }
}

// GT[set][t][c][i] = G[set][i][c][t], from the [set][t][i][c] image the CUDA-core path keeps.
__global__ void pack_gt_kernel(const __nv_bfloat16* gp, __nv_bfloat16* gt, int M, int C) {
    __shared__ __nv_bfloat16 tile[32][33];
    const int64_t plane = (int64_t)blockIdx.z * M * C;      // (set, tap)
    const int i0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) tile[r][threadIdx.x] = gp[plane + (int64_t)(i0 + r) * C + c0 + threadIdx.x];
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) gt[plane + (int64_t)(c0 + r) * M + i0 + threadIdx.x] = tile[threadIdx.x][r];
}

// One block per (unit, slot) row: dA = [R>0] (dw - <dw, w>) / s with w = R / s (Eq. 7 reversed), in bf16,
// zero from column S up to the row stride; R comes from the recompute in bf16 (rows of Sp, zero beyond S);
// dbias += sum of dA.
__global__ void __launch_bounds__(256) da_row_kernel(BwdStep p, const float* dw, __nv_bfloat16* dab, const __nv_bfloat16* rb, int Sp) {
    __shared__ float red[8];
    const int64_t row = blockIdx.x;                          // u * M + i
    const float* dwr = dw + row * Sp;
    const __nv_bfloat16* Rr = rb + row * Sp;
    const float inv_s = 1.f / p.s[row];
    float acc = 0.f;
    for (int j = threadIdx.x; j < p.S; j += 256) acc = fmaf(__bfloat162float(Rr[j]), dwr[j], acc);
    for (int of = 16; of > 0; of >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, of);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    float dot = 0.f;
    for (int w = 0; w < 8; ++w) dot += red[w];
    dot *= inv_s;                                            // <dw, w>
    float bsum = 0.f;
    for (int j = threadIdx.x; j < Sp; j += 256) {
        float da = 0.f;
        if (j < p.S && __bfloat162float(Rr[j]) > 0.f) da = (dwr[j] - dot) * inv_s;
        dab[row * Sp + j] = __float2bfloat16_rn(da);
        bsum += da;
    }
    if (p.dbias) {
        __syncthreads();
        for (int of = 16; of > 0; of >>= 1) bsum += __shfl_xor_sync(0xffffffffu, bsum, of);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = bsum;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;
            for (int w = 0; w < 8; ++w) t += red[w];
            const int u = (int)(row / p.M), i = (int)(row % p.M);
            atomicAdd(p.dbias + (p.weights_per_head ? (u % p.heads) * p.M : 0) + i, t);
        }
    }
}

// dAT[u][j][i] = dAb[u][i][j]: 64 x 64 tiles through shared memory.
__global__ void __launch_bounds__(256) transpose_kernel(const __nv_bfloat16* in, __nv_bfloat16* out, int M, int Sp) {
    __shared__ __nv_bfloat16 tile[64][66];
    const int u = blockIdx.z, i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    for (int r = ty; r < 64; r += 4) {
        const int j = j0 + tx;
        tile[r][tx] = j < Sp ? in[((int64_t)u * M + i0 + r) * Sp + j] : __float2bfloat16_rn(0.f);
    }
    __syncthreads();
    for (int r = ty; r < 64; r += 4) {
        const int j = j0 + r;
        if (j < Sp) out[((int64_t)u * Sp + j) * M + i0 + tx] = tile[tx][r];
    }
}

// ------------------------------------------------------------------ GEMM set-up helpers
struct Tensor4 {
    const void* base;
    uint64_t d[4];      // extents, innermost first
    uint64_t s[3];      // byte strides of extents 1..3
};
bool operand(gemm::Operand& O, const Tensor4& t, bool mn_major) {
    O = gemm::Operand{};
    O.mn_major = mn_major ? 1 : 0;
    uint64_t s[3] = {t.s[0], t.s[1], t.s[2]};
    // an extent of 1 never uses its stride: give it a harmless one
    if (t.d[2] <= 1) s[1] = s[0] * std::max<uint64_t>(t.d[1], 1);
    if (t.d[3] <= 1) s[2] = s[1] * std::max<uint64_t>(t.d[2], 1);
    return gemm::make_map(&O.map, t.base, t.d, s, mn_major);
}
// [batch, heads, tokens, 128] view of the caller with `tokens` valid rows
Tensor4 of_view(const View& v, int tokens, int heads, int batch) {
    return Tensor4{v.ptr, {(uint64_t)kD, (uint64_t)tokens, (uint64_t)heads, (uint64_t)batch},
                   {(uint64_t)v.st * 2, (uint64_t)v.sh * 2, (uint64_t)v.sb * 2}};
}
gemm::Params base_params(lococo_handle* h) {
    gemm::Params P{};
    P.n_inner = P.s_inner = P.z_inner = 1 << 30;
    P.out_n_inner = 1 << 30;
    P.out_n_in = 1;
    P.splits = 1;
    P.alpha = 1.f;
    P.status = reinterpret_cast<int*>(h->ws + h->off_status);
    return P;
}

}  // namespace

bool tensor_backward_supported(const lococo_handle* h) {
    const lococo_config& c = h->cfg;
    return h->use_tensor && c.dtype == LOCOCO_BF16 && c.head_dim == kD && c.M % 128 == 0 && gemm::encode_tiled() != nullptr;
}

size_t tensor_backward_scratch_bytes(const lococo_handle* h, int B) { return layout_of(h, B).total; }

int tensor_backward_prepare(lococo_handle* h, int B, char* sc, cudaStream_t st) {
    const lococo_config& c = h->cfg;
    const Layout L = layout_of(h, B);
    const int sets = c.weights_per_head ? c.heads : 1;
    pack_gt_kernel<<<dim3(c.c_in / 32, c.M / 32, sets * c.k), dim3(32, 8), 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(h->ws + h->off_gpack), reinterpret_cast<__nv_bfloat16*>(sc + L.gt), c.M, c.c_in);
    return launched() ? 1 : -1;
}

int tensor_backward_pack(lococo_handle* h, const BwdStep& p, int B, char* sc, cudaStream_t st) {
    const Layout L = layout_of(h, B);
    pack_x_kernel<<<dim3(std::min((L.Sp2 + 7) / 8, 512), p.units), 256, 0, st>>>(p, reinterpret_cast<__nv_bfloat16*>(sc + L.xpad), L.Sp2,
                                                                                  (p.k - 1) / 2);
    return launched() ? 1 : -1;
}

int tensor_backward_compress(lococo_handle* h, const BwdStep& p, const CompressParams& fwd, int B, char* sc, cudaStream_t st) {
    const Layout L = layout_of(h, B);
    const int U = p.units, H = p.heads, M = p.M, S = p.S, C = p.c_in, k = p.k, pad = (k - 1) / 2;
    const int sets = p.weights_per_head ? H : 1, in_set = U / sets;
    __nv_bfloat16* xpad = reinterpret_cast<__nv_bfloat16*>(sc + L.xpad);
    __nv_bfloat16* gkv = reinterpret_cast<__nv_bfloat16*>(sc + L.gkv);
    __nv_bfloat16* gkv_lo = reinterpret_cast<__nv_bfloat16*>(sc + L.gkv_lo);
    if (L.gs_lo - L.gs != L.gkv_lo - L.gkv) return -1;
    __nv_bfloat16* wb = reinterpret_cast<__nv_bfloat16*>(sc + L.wb);
    __nv_bfloat16* dab = reinterpret_cast<__nv_bfloat16*>(sc + L.dab);
    __nv_bfloat16* dat = reinterpret_cast<__nv_bfloat16*>(sc + L.dat);
    float* dw = reinterpret_cast<float*>(sc + L.dw);
    int n = 0;

    // R and s of the forward, by the forward's kernel; its cache output goes to a dummy
    CompressParams f = fwd;
    f.k_out = View{sc + L.dummy_k, (int64_t)H * M * kD, (int64_t)M * kD, kD};
    f.v_out = View{sc + L.dummy_v, (int64_t)H * M * kD, (int64_t)M * kD, kD};
    f.W_out = nullptr;
    f.R16 = wb;             // R in bf16 (exact: the forward rounds it), rows of Sp
    f.R16_stride = L.Sp;
    f.prof = nullptr;
    const int r = tensor_compress(h, f, st);
    if (r < 0) return -1;
    n += r;

    pack_g_kernel<<<std::min<int64_t>(((int64_t)U * M * 256 + 255) / 256, 4096), 256, 0, st>>>(p.gK, p.gV, p.s, gkv, gkv_lo, reinterpret_cast<__nv_bfloat16*>(sc + L.gs),
                                                                                       reinterpret_cast<__nv_bfloat16*>(sc + L.gs_lo), (int64_t)U * M);
    if (!launched()) return -1;
    ++n;

    const Tensor4 t_xpad{xpad, {256, (uint64_t)L.Sp2, (uint64_t)U, 1}, {512, (uint64_t)L.Sp2 * 512, (uint64_t)U * L.Sp2 * 512}};
    const int m_tiles = M / 128, s_tiles = (S + 127) / 128;

    const uint64_t part_stride = L.gkv_lo - L.gkv;          // value and remainder lie the same distance apart in both pairs
    {   // dw[u] = gKV[u] Xcat[u]^T: one K loop over the value's and then the remainder's 2d channels
        gemm::Params G = base_params(h);
        const Tensor4 t_g2{gkv, {256, (uint64_t)M, (uint64_t)U, 2}, {512, (uint64_t)M * 512, part_stride}};
        if (!operand(G.A, t_g2, false) || !operand(G.B, t_xpad, false)) return -1;
        G.s_inner = 4;
        G.A.c[0].si = 64; G.A.c[1].tm = 128; G.A.c[2].zi = 1; G.A.c[3].so = 1;
        G.B.c[0].si = 64; G.B.c[1].c0 = pad; G.B.c[1].tni = 128; G.B.c[2].zi = 1;
        G.steps = 8;
        G.out = dw; G.out_zi = (int64_t)M * L.Sp; G.out_m = L.Sp;
        G.M = M; G.N = S; G.mode = gemm::kStoreF32;
        if (!gemm::launch(G, m_tiles, s_tiles, U, st)) return -1;
        ++n;
    }
    da_row_kernel<<<U * M, 256, 0, st>>>(p, dw, dab, wb, L.Sp);
    transpose_kernel<<<dim3((L.Sp + 63) / 64, M / 64, U), 256, 0, st>>>(dab, dat, M, L.Sp);
    if (!launched()) return -1;
    n += 2;

    const Tensor4 t_wb{wb, {(uint64_t)L.Sp, (uint64_t)M, (uint64_t)U, 1}, {(uint64_t)L.Sp * 2, (uint64_t)M * L.Sp * 2, (uint64_t)U * M * L.Sp * 2}};
    const Tensor4 t_dab{dab, {(uint64_t)L.Sp, (uint64_t)M, (uint64_t)U, 1}, {(uint64_t)L.Sp * 2, (uint64_t)M * L.Sp * 2, (uint64_t)U * M * L.Sp * 2}};
    {   // dX[u] += R[u]^T (g / s)[u]   (columns 0-127 -> dX_K, 128-255 -> dX_V); K loop over the slots, twice
        gemm::Params G = base_params(h);
        const Tensor4 t_gs2{sc + L.gs, {256, (uint64_t)M, (uint64_t)U, 2}, {512, (uint64_t)M * 512, part_stride}};
        if (!operand(G.A, t_wb, true) || !operand(G.B, t_gs2, true)) return -1;
        G.s_inner = M / 64;
        G.A.c[0].tm = 128; G.A.c[1].si = 64; G.A.c[2].zi = 1;
        G.B.c[0].tni = 128; G.B.c[1].si = 64; G.B.c[2].zi = 1; G.B.c[3].so = 1;
        G.steps = 2 * (M / 64);
        G.out = p.dXK; G.out_zi = (int64_t)S * kD; G.out_m = kD;
        G.out_n_inner = kD; G.out_n_in = 1; G.out_n_out = p.dXV - p.dXK;
        G.M = S; G.N = 256; G.mode = gemm::kAddF32;
        if (!gemm::launch(G, s_tiles, 2, U, st)) return -1;
        ++n;
    }
    {   // dG[set] += sum over the set's units and positions of dA (*) Z; n = t * C + c
        gemm::Params G = base_params(h);
        const Tensor4 t_z{xpad, {(uint64_t)C, (uint64_t)S, (uint64_t)k, (uint64_t)U}, {512, 512, (uint64_t)L.Sp2 * 512}};
        if (!operand(G.A, t_dab, false) || !operand(G.B, t_z, true)) return -1;
        const int unit_so = p.weights_per_head ? H : 1, unit_zi = p.weights_per_head ? 1 : 0;
        G.s_inner = (S + 63) / 64;
        G.n_inner = C / 128;
        G.A.c[0].si = 64; G.A.c[1].tm = 128; G.A.c[2].so = unit_so; G.A.c[2].zi = unit_zi;
        G.B.c[0].tni = 128; G.B.c[1].si = 64; G.B.c[2].tno = 1; G.B.c[3].so = unit_so; G.B.c[3].zi = unit_zi;
        G.steps = in_set * G.s_inner;
        const int tiles = m_tiles * (k * C / 128) * sets;
        // K splits: fill whole waves of the 2 x 148 CTA slots (the split partials meet in atomics)
        double best = 0.0;
        for (int sp = 1; sp <= 16 && (sp == 1 || G.steps / sp >= 32); ++sp) {   // a split keeps at least 32 K steps
            const int ctas = tiles * sp, waves = (ctas + 295) / 296;
            const double fill = (double)ctas / (waves * 296.0) - 0.002 * sp;
            if (fill > best) { best = fill; G.splits = sp; }
        }
        G.out = p.dG; G.out_zi = (int64_t)M * C * k; G.out_m = (int64_t)C * k;
        G.out_n_inner = C; G.out_n_in = k; G.out_n_out = 1;
        G.M = M; G.N = k * C; G.mode = gemm::kAtomicF32;
        if (!gemm::launch(G, m_tiles, k * C / 128, sets, st)) return -1;
        ++n;
    }
    {   // dZ (into dX): sum over taps of shift_t(dA^T) G_t; a tap is a row offset of the box of dA^T
        gemm::Params G = base_params(h);
        const Tensor4 t_dat{dat, {(uint64_t)M, (uint64_t)S, (uint64_t)U, 1}, {(uint64_t)M * 2, (uint64_t)L.Sp * M * 2, (uint64_t)U * L.Sp * M * 2}};
        const Tensor4 t_gt{sc + L.gt, {(uint64_t)M, (uint64_t)C, (uint64_t)k, (uint64_t)sets},
                           {(uint64_t)M * 2, (uint64_t)C * M * 2, (uint64_t)k * C * M * 2}};
        if (!operand(G.A, t_dat, false) || !operand(G.B, t_gt, false)) return -1;
        G.s_inner = M / 64;
        G.z_inner = H;
        G.A.c[0].si = 64; G.A.c[1].c0 = pad; G.A.c[1].tm = 128; G.A.c[1].so = -1; G.A.c[2].zi = 1; G.A.c[2].zo = H;
        G.B.c[0].si = 64; G.B.c[1].tni = 128; G.B.c[2].so = 1; G.B.c[3].zi = p.weights_per_head ? 1 : 0;
        G.steps = k * (M / 64);
        G.out = p.dXK; G.out_zi = (int64_t)S * kD; G.out_zo = (int64_t)H * S * kD; G.out_m = kD;
        G.out_n_inner = kD; G.out_n_in = 1; G.out_n_out = p.dXV - p.dXK;
        G.M = S; G.N = C; G.mode = gemm::kAddF32;
        if (!gemm::launch(G, s_tiles, C / 128, U, st)) return -1;
        ++n;
    }
    return n;
}

int tensor_backward_attention(lococo_handle* h, const BwdStep& p, int B, char* sc, cudaStream_t st) {
    const Layout L = layout_of(h, B);
    const int U = p.units, H = p.heads, batch = U / H, S = p.S, pad = (p.k - 1) / 2;
    __nv_bfloat16* xpad = reinterpret_cast<__nv_bfloat16*>(sc + L.xpad);
    __nv_bfloat16* pb = reinterpret_cast<__nv_bfloat16*>(sc + L.pb);
    __nv_bfloat16* dsb = reinterpret_cast<__nv_bfloat16*>(sc + L.dsb);
    const Tensor4 t_xpad{xpad, {256, (uint64_t)L.Sp2, (uint64_t)U, 1}, {512, (uint64_t)L.Sp2 * 512, (uint64_t)U * L.Sp2 * 512}};
    const Tensor4 t_q = of_view(p.q, p.b, H, batch), t_do = of_view(p.d_o, p.b, H, batch);
    const int s_tiles = (S + 127) / 128;
    int n = 0;
    for (int q0 = 0; q0 < p.b; q0 += L.QB) {
        const int qb = std::min(L.QB, p.b - q0), q_tiles = (qb + 127) / 128;
        const int Sv = std::min(S, p.c + q0 + qb);          // keys any query of the block can see
        const int sv_tiles = (Sv + 127) / 128;
        // P = exp(scale Q X_K^T - lse) and dS = scale P (dO X_V^T - delta): ONE launch computes both products
        // of a tile into two accumulators and applies the softmax and its gradient to them, under the causal
        // mask; only bf16 P and dS reach memory
        {
            gemm::Params G = base_params(h);
            if (!operand(G.A, t_q, false) || !operand(G.B, t_xpad, false) || !operand(G.A2, t_do, false) || !operand(G.B2, t_xpad, false))
                return -1;
            G.z_inner = H;
            for (int which = 0; which < 2; ++which) {
                gemm::Operand& A = which ? G.A2 : G.A;
                gemm::Operand& Bo = which ? G.B2 : G.B;
                A.c[0].si = 64; A.c[1].c0 = q0; A.c[1].tm = 128; A.c[2].zi = 1; A.c[3].zo = 1;
                Bo.c[0].c0 = which * kD; Bo.c[0].si = 64; Bo.c[1].c0 = pad; Bo.c[1].tni = 128; Bo.c[2].zi = 1; Bo.c[2].zo = H;
            }
            G.steps = 2;
            G.out = pb; G.out2 = dsb;
            G.out_zi = (int64_t)L.QB * L.Sp; G.out_zo = (int64_t)H * L.QB * L.Sp; G.out_m = L.Sp;
            G.M = qb; G.N = Sv;
            G.causal_tiles = 1; G.causal_c = p.c + q0;
            G.mode = gemm::kPairBF16; G.alpha = p.scale; G.scale2 = p.scale * 1.4426950408889634f;
            G.rowvec = p.lse + q0; G.rowvec_z = p.lse_stride;
            G.rowvec2 = p.delta + q0; G.rowvec2_z = p.b;
            if (!gemm::launch(G, q_tiles, sv_tiles, U, st)) return -1;
            ++n;
        }
        const Tensor4 t_pb{pb, {(uint64_t)Sv, (uint64_t)qb, (uint64_t)U, 1}, {(uint64_t)L.Sp * 2, (uint64_t)L.QB * L.Sp * 2, (uint64_t)U * L.QB * L.Sp * 2}};
        const Tensor4 t_dsb{dsb, {(uint64_t)Sv, (uint64_t)qb, (uint64_t)U, 1}, {(uint64_t)L.Sp * 2, (uint64_t)L.QB * L.Sp * 2, (uint64_t)U * L.QB * L.Sp * 2}};
        for (int which = 0; which < 2; ++which) {           // dX_V += P^T dO, dX_K += dS^T Q
            gemm::Params G = base_params(h);
            if (!operand(G.A, which ? t_dsb : t_pb, true) || !operand(G.B, which ? t_q : t_do, true)) return -1;
            G.z_inner = H;
            G.A.c[0].tm = 128; G.A.c[1].si = 64; G.A.c[2].zi = 1; G.A.c[2].zo = H;
            G.B.c[0].tni = 128; G.B.c[1].c0 = q0; G.B.c[1].si = 64; G.B.c[2].zi = 1; G.B.c[3].zo = 1;
            G.steps = (qb + 63) / 64;
            G.k_lo_on = 1; G.k_lo_c0 = -(p.c + q0);          // query rows that cannot see this key tile contribute nothing
            G.out = which ? p.dXK : p.dXV; G.out_zi = (int64_t)S * kD; G.out_zo = (int64_t)H * S * kD; G.out_m = kD;
            G.M = Sv; G.N = kD; G.mode = gemm::kAddF32;
            if (!gemm::launch(G, sv_tiles, 1, U, st)) return -1;
            ++n;
        }
        {   // dQ = dS X_K
            gemm::Params G = base_params(h);
            if (!operand(G.A, t_dsb, false) || !operand(G.B, t_xpad, true)) return -1;
            G.z_inner = H;
            G.A.c[0].si = 64; G.A.c[1].tm = 128; G.A.c[2].zi = 1; G.A.c[2].zo = H;
            G.B.c[0].tni = 128; G.B.c[1].c0 = pad; G.B.c[1].si = 64; G.B.c[2].zi = 1; G.B.c[2].zo = H;
            G.steps = (Sv + 63) / 64;
            G.k_hi_on = 1; G.k_hi_c0 = p.c + q0 + 128;       // keys beyond the last query of the tile are masked
            G.out = reinterpret_cast<__nv_bfloat16*>(p.dq.ptr) + (int64_t)q0 * p.dq.st;
            G.out_zi = p.dq.sh; G.out_zo = p.dq.sb; G.out_m = p.dq.st;
            G.M = qb; G.N = kD; G.mode = gemm::kStoreBF16;
            if (!gemm::launch(G, q_tiles, 1, U, st)) return -1;
            ++n;
        }
    }
    (void)s_tiles;
    return n;
}

}  // namespace lococo
