// Backward pass of Algorithm 2 on the tensor cores (bf16 storage, d = 128, M a multiple of 128).
// Every contraction of one reversed step is a launch of the batched GEMM of gemm_tc.cuh on operands
// that small packing kernels lay out once per step:
//   cache update (Eq. 4-7 reversed)
//     R, s        recomputed by the forward's own tcgen05 conv kernel (R left in place)
//     dw          = [gK | gV] [X_K | X_V]^T                          per unit, K = 2d
//     dA          row kernel: dA = [R>0] (dw - <dw, w>_row) / s with w = R / s, rounded to bf16, written in both orientations
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

// dA = [R>0] (dw - <dw, w>) / s with w = R / s (Eq. 7 reversed), rounded to bf16, in both orientations: dAb[u][i][j]
// (rows of Sp, zero from column S on) and dAT[u][j][i]. One block per 16 consecutive slots of a unit, so that a
// thread's piece of the transposed copy is 16 slots = one full 32-byte sector. R comes from the recompute in bf16
// (rows of Sp, zero beyond S); dbias += sum of dA.
constexpr int kDaRows = 16;
__global__ void __launch_bounds__(256) da_rows_kernel(BwdStep p, const float* dw, __nv_bfloat16* dab, __nv_bfloat16* dat, const __nv_bfloat16* rb, int Sp) {
    __shared__ float dots[kDaRows], bias_sum[kDaRows];
    const int blocks_per_unit = p.M / kDaRows;
    const int u = blockIdx.x / blocks_per_unit, i0 = (blockIdx.x % blocks_per_unit) * kDaRows;
    const int64_t row0 = (int64_t)u * p.M + i0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // <dw, w> of the 16 rows: two rows per warp
    for (int r = warp; r < kDaRows; r += 8) {
        const float* dwr = dw + (row0 + r) * Sp;
        const __nv_bfloat16* Rr = rb + (row0 + r) * Sp;
        float acc = 0.f;
        for (int j = lane; j < p.S; j += 32) acc = fmaf(__bfloat162float(Rr[j]), dwr[j], acc);
        for (int of = 16; of > 0; of >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, of);
        if (lane == 0) { dots[r] = acc / p.s[row0 + r]; bias_sum[r] = 0.f; }
    }
    __syncthreads();
    float inv_s[kDaRows], dot[kDaRows], bsum[kDaRows];
#pragma unroll
    for (int r = 0; r < kDaRows; ++r) { inv_s[r] = 1.f / p.s[row0 + r]; dot[r] = dots[r]; bsum[r] = 0.f; }
    // a thread takes a position j and all 16 rows: the rows' reads and writes are 2- or 4-byte pieces of lines the
    // whole warp covers (consecutive j), the transposed write is 32 bytes
    for (int j = threadIdx.x; j < Sp; j += 256) {
        __align__(16) __nv_bfloat16 col[kDaRows];
        float rv[kDaRows], dwv[kDaRows];
#pragma unroll
        for (int r = 0; r < kDaRows; ++r) {          // all 32 loads first: they do not depend on one another
            rv[r] = __bfloat162float(rb[(row0 + r) * Sp + j]);
            dwv[r] = dw[(row0 + r) * Sp + j];
        }
#pragma unroll
        for (int r = 0; r < kDaRows; ++r) {
            const float da = (j < p.S && rv[r] > 0.f) ? (dwv[r] - dot[r]) * inv_s[r] : 0.f;
            col[r] = __float2bfloat16_rn(da);
            dab[(row0 + r) * Sp + j] = col[r];
            bsum[r] += da;
        }
        uint4* dst = reinterpret_cast<uint4*>(dat + ((int64_t)u * Sp + j) * p.M + i0);
        dst[0] = *reinterpret_cast<const uint4*>(col);
        dst[1] = *reinterpret_cast<const uint4*>(col + 8);
    }
    if (p.dbias) {
#pragma unroll
        for (int r = 0; r < kDaRows; ++r) {
            float t = bsum[r];
            for (int of = 16; of > 0; of >>= 1) t += __shfl_xor_sync(0xffffffffu, t, of);
            if (lane == 0) atomicAdd(&bias_sum[r], t);
        }
        __syncthreads();
        if (threadIdx.x < kDaRows)
            atomicAdd(p.dbias + (p.weights_per_head ? (u % p.heads) * p.M : 0) + i0 + threadIdx.x, bias_sum[threadIdx.x]);
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


// ------------------------------------------------------------------ Eq. 1 reversed, keys' side, fused
// One CTA owns a tile of 128 keys of one unit and walks over the tiles of 64 queries that can see it. Per query tile:
//   S^T = X_K Q^T and dP^T = X_V dO^T           (keys on the TMEM lanes, queries on the columns)
//   P^T = exp(scale S^T - lse), dS^T = scale P^T (dP^T - delta), under the causal mask, in registers (P in fp32);
//         both go to shared memory in bf16 as MMA A operands, dS^T also to global memory for dQ = dS X_K
//   dX_V += P^T dO, dX_K += dS^T Q                accumulated in TMEM over all query tiles, added to memory at the end
// so P never reaches memory and dS is written once. Three roles meet at mbarriers: one lane drives the tensor copy
// engine (keys and values once, then Q / dO tiles through two stages), one lane issues the MMAs (the score products of
// tile t+1 are queued behind the gradient products of tile t), sixteen warps turn scores into P^T and dS^T (that
// part is bound by instruction issue: about a microsecond per tile with eight warps).
// TMEM: S^T x2 (64 columns each), dP^T x2, dX_V, dX_K (128 each) = 512 columns.
namespace fused {

using namespace tc;

constexpr int kEpiWarps = 16;             // four warps per TMEM lane quarter, 16 of a tile's 64 queries each
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kMmaThread = kEpiThreads, kLoadThread = kEpiThreads + 32;
constexpr int kThreads = kEpiThreads + 64;
constexpr uint32_t kKvTile = 32768;       // 128 rows x 128 channels: two 64-channel halves of 16 KB (128-byte swizzle)
constexpr uint32_t kQTile = 16384;        // 64 rows x 128 channels: two halves of 8 KB
constexpr uint32_t kPTile = 16384;        // 128 keys x 64 queries, bf16: [8-query group][128 rows][8 queries]
constexpr int kQStages = 3;              // Q / dO stages: a stage is held from its score products to its gradient products, and a tile takes about a
                                         // microsecond to arrive, so two stages leave the tensor pipe waiting for loads
constexpr uint32_t kSmem = 2 * kKvTile + kQStages * 2 * kQTile + 2 * 2 * kPTile + 2 * 128 * 4 + 256 + 1024;

struct alignas(64) Params {
    CUtensorMap map_x;            // packed [unit][pad + position][K 128 | V 128], boxes of 128 rows x 64 channels
    CUtensorMap map_q, map_do;    // [batch, heads, tokens, 128] views, boxes of 64 rows x 64 channels
    const float* lse;             // log-sum-exp of the forward, first query of the block; lse_z: unit stride
    const float* delta;           // <dO, O> per query, first query of the block
    int64_t lse_z, delta_z;
    __nv_bfloat16* ds_t;          // dS^T [unit][key][query of the block], row stride ds_row, unit stride ds_z
    int64_t ds_z;
    int ds_row;
    float* dXK;                   // [unit][S][128] fp32, += ; dXV likewise
    float* dXV;
    int heads, S, c, pad;
    int q0, qb, b;                // first query of the block, queries in the block, chunk length
    float scale, scale2;          // softmax scale, and scale * log2 e
    int* status;
};

__global__ void __launch_bounds__(kThreads, 1) attn_bwd_kv_kernel(const __grid_constant__ Params P) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* k_ptr = smem;
    uint8_t* v_ptr = k_ptr + kKvTile;
    uint8_t* qd_ptr = v_ptr + kKvTile;                 // stage x: [Q | dO]
    uint8_t* p_ptr = qd_ptr + kQStages * 2 * kQTile;   // buffer x: [P^T | dS^T]
    float* vec = reinterpret_cast<float*>(p_ptr + 2 * 2 * kPTile);   // buffer x: [64 lse * log2 e | 64 delta]
    uint64_t* bars = reinterpret_cast<uint64_t*>(vec + 2 * 128);
    volatile int* failed = reinterpret_cast<volatile int*>(bars + 16);
    const uint32_t ks = smem_u32(k_ptr), vs = smem_u32(v_ptr), qds = smem_u32(qd_ptr), ps = smem_u32(p_ptr);
    const uint32_t bar0 = smem_u32(bars);
    auto qd_full = [&](int x) { return bar0 + 8 * x; };           // loader -> MMA: Q, dO tile staged (three stages)
    auto qd_free = [&](int x) { return bar0 + 24 + 8 * x; };      // MMA -> loader: gradient products have read the stage
    auto s_full = [&](int x) { return bar0 + 48 + 8 * x; };       // MMA -> warps: S^T, dP^T in TMEM
    auto s_free = [&](int x) { return bar0 + 64 + 8 * x; };       // warps -> MMA: S^T, dP^T read
    auto p_full = [&](int x) { return bar0 + 80 + 8 * x; };       // warps -> MMA: P^T, dS^T written
    auto g_done = [&](int x) { return bar0 + 96 + 8 * x; };       // MMA -> warps: gradient products have read P^T, dS^T
    const uint32_t kv_full = bar0 + 112, acc_done = bar0 + 120;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int jt = blockIdx.x, u = blockIdx.y;
    const int n = u / P.heads, h = u % P.heads;
    const int j0 = jt * 128;

    if (tid == kMmaThread) {
        for (int x = 0; x < kQStages; ++x) {
            mbar_init(qd_full(x), 1);
            mbar_init(qd_free(x), 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(s_full(x), 1);
            mbar_init(s_free(x), kEpiThreads);
            mbar_init(p_full(x), kEpiThreads);
            mbar_init(g_done(x), 1);
        }
        mbar_init(kv_full, 1);
        mbar_init(acc_done, 1);
        *failed = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // query tiles (64 rows) of the block that see a key of this tile; whole pairs of tiles, because dQ = dS X_K works in
    // tiles of 128 queries and reads what is written here, zeros included
    const int T = (P.qb + 63) / 64;
    const int first = 2 * (max(0, j0 - P.c - P.q0) / 128);
    const bool any = first < T && j0 < P.S;

    if (tid == kLoadThread && any) {
        // ---------------- loader
        mbar_expect_tx(kv_full, 2 * kKvTile);
        for (int x = 0; x < 4; ++x)      // K channels 0-63, 64-127, V channels 0-63, 64-127
            tma_load_4d(ks + x * (kKvTile / 2), &P.map_x, 64 * x, P.pad + j0, u, 0, kv_full);
#pragma unroll 1
        for (int t = first; t < T; ++t) {
            const int x = (t - first) % kQStages, use = (t - first) / kQStages;
            if (use >= 1) mbar_wait(qd_free(x), (use - 1) & 1, P.status, failed, 40);
            mbar_expect_tx(qd_full(x), 2 * kQTile);
            const uint32_t dst = qds + x * 2 * kQTile;
            const int row = P.q0 + 64 * t;
            tma_load_4d(dst, &P.map_q, 0, row, h, n, qd_full(x));
            tma_load_4d(dst + kQTile / 2, &P.map_q, 64, row, h, n, qd_full(x));
            tma_load_4d(dst + kQTile, &P.map_do, 0, row, h, n, qd_full(x));
            tma_load_4d(dst + kQTile + kQTile / 2, &P.map_do, 64, row, h, n, qd_full(x));
        }
    } else if (tid == kMmaThread && any) {
        // ---------------- MMA issuer
        const uint32_t idesc_s = instr_desc_bf16(64, false, false);
        const uint32_t idesc_g = instr_desc_bf16(128, false, true);
        const uint64_t ka = smem_desc_sw128(ks, 16, 1024), va = smem_desc_sw128(vs, 16, 1024);
        auto issue_grad = [&](int t) {
            const int x = (t - first) & 1, use = (t - first) >> 1, sx = (t - first) % kQStages;
            mbar_wait(p_full(x), use & 1, P.status, failed, 41);
            tc_fence_after();
            const uint32_t q_addr = qds + sx * 2 * kQTile, pt = ps + x * 2 * kPTile;
            const uint64_t pa = smem_desc(pt, 2048, 128), da = smem_desc(pt + kPTile, 2048, 128);
            const uint64_t qb_mn = smem_desc_sw128(q_addr, kQTile / 2, 1024), dob_mn = smem_desc_sw128(q_addr + kQTile, kQTile / 2, 1024);
            // 16 queries per step: two 8-query groups of the A operand, two 8-row groups of the B operand
            umma_ss_k4(tmem + 256, pa, dob_mn, 256u, 128u, idesc_g, t != first);
            umma_ss_k4(tmem + 384, da, qb_mn, 256u, 128u, idesc_g, t != first);
            umma_commit(g_done(x));
            umma_commit(qd_free(sx));
        };
        mbar_wait(kv_full, 0, P.status, failed, 42);
#pragma unroll 1
        for (int t = first; t < T; ++t) {
            const int x = (t - first) & 1, use = (t - first) >> 1, sx = (t - first) % kQStages;
            mbar_wait(qd_full(sx), ((t - first) / kQStages) & 1, P.status, failed, 43);
            if (use >= 1) mbar_wait(s_free(x), (use - 1) & 1, P.status, failed, 44);
            tc_fence_after();
            const uint32_t q_addr = qds + sx * 2 * kQTile;
            const uint64_t qk = smem_desc_sw128(q_addr, 16, 1024), dok = smem_desc_sw128(q_addr + kQTile, 16, 1024);
            // 128 channels: 32 bytes per 16-channel step inside a 128-byte row, then the second 64-channel half of each tile
            umma_ss_k4(tmem + x * 64, ka, qk, 2u, 2u, idesc_s, 0);
            umma_ss_k4(tmem + x * 64, ka + ((kKvTile / 2) >> 4), qk + ((kQTile / 2) >> 4), 2u, 2u, idesc_s, 1);
            umma_ss_k4(tmem + 128 + x * 64, va, dok, 2u, 2u, idesc_s, 0);
            umma_ss_k4(tmem + 128 + x * 64, va + ((kKvTile / 2) >> 4), dok + ((kQTile / 2) >> 4), 2u, 2u, idesc_s, 1);
            umma_commit(s_full(x));
            if (t > first) issue_grad(t - 1);
        }
        issue_grad(T - 1);
        umma_commit(acc_done);
    }
    if (warp < kEpiWarps && any) {
        // ---------------- P^T and dS^T: a thread owns one key (TMEM lane) and 16 of the tile's 64 queries
        const int rl = (warp & 3) * 32 + lane, part = warp >> 2;
        const int j = j0 + rl;
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        __nv_bfloat16* ds_row = P.ds_t + (int64_t)u * P.ds_z + (int64_t)j * P.ds_row;
        // per-query vectors of a tile (lse * log2 e, delta): threads 0-127 fetch one value each, a tile ahead, so that
        // the load's latency is not part of an iteration
        auto fetch = [&](int t) {
            const int q = 64 * t + (tid & 63);                       // query within the block
            if (tid >= 128 || t >= T || q >= P.qb) return 0.f;
            return tid < 64 ? P.lse[(int64_t)u * P.lse_z + q] * 1.4426950408889634f : P.delta[(int64_t)u * P.delta_z + q];
        };
        float next_vec = fetch(first);
#pragma unroll 1
        for (int t = first; t < T; ++t) {
            const int x = (t - first) & 1, use = (t - first) >> 1;
            float* vb = vec + x * 128;
            if (tid < 128) vb[tid] = next_vec;
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
            next_vec = fetch(t + 1);
            mbar_wait(s_full(x), use & 1, P.status, failed, 45);
            tc_fence_after();
            uint32_t sv[16], dv[16];
            tmem_ld16(lane_base + x * 64 + part * 16, sv);
            tmem_ld16(lane_base + 128 + x * 64 + part * 16, dv);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(s_free(x));
            if (use >= 1) mbar_wait(g_done(x), (use - 1) & 1, P.status, failed, 46);      // the P^T, dS^T buffer is free again
            const int qc0 = 64 * t + part * 16;                      // first of this thread's queries, within the block
            // key j is seen by query r of the chunk when j < c + r + 1
            const int lim = j - P.c - P.q0;                          // visible: query (within the block) >= lim
            uint8_t* pdst = p_ptr + x * 2 * kPTile + rl * 16;
            // tiles that neither the causal limit nor the end of the keys or queries cuts need no tests (the common case)
            const bool whole = j0 + 128 <= P.S && 64 * t + 64 <= P.qb && j0 + 127 - P.c - P.q0 <= 64 * t;
            const float4* lv = reinterpret_cast<const float4*>(vb + part * 16);
            const float4* dl = reinterpret_cast<const float4*>(vb + 64 + part * 16);
#pragma unroll
            for (int e = 0; e < 16; e += 8) {
                const float4 la = lv[e >> 2], lb = lv[(e >> 2) + 1], da = dl[e >> 2], db = dl[(e >> 2) + 1];
                const float ls[8] = {la.x, la.y, la.z, la.w, lb.x, lb.y, lb.z, lb.w};
                const float de[8] = {da.x, da.y, da.z, da.w, db.x, db.y, db.z, db.w};
                float pv[8], dsv[8];
#pragma unroll
                for (int y = 0; y < 8; ++y) {
                    pv[y] = exp2f(fmaf(__uint_as_float(sv[e + y]), P.scale2, -ls[y]));
                    if (!whole) {
                        const int qa = qc0 + e + y;
                        if (!(j < P.S && qa < P.qb && qa >= lim)) pv[y] = 0.f;
                    }
                    dsv[y] = pv[y] * (__uint_as_float(dv[e + y]) - de[y]) * P.scale;
                }
                const uint4 pk = make_uint4(pack_bf16(pv[0], pv[1]), pack_bf16(pv[2], pv[3]), pack_bf16(pv[4], pv[5]), pack_bf16(pv[6], pv[7]));
                const uint4 dk = make_uint4(pack_bf16(dsv[0], dsv[1]), pack_bf16(dsv[2], dsv[3]), pack_bf16(dsv[4], dsv[5]), pack_bf16(dsv[6], dsv[7]));
                const uint32_t g = (uint32_t)((part * 16 + e) >> 3) * 2048u;
                *reinterpret_cast<uint4*>(pdst + g) = pk;
                *reinterpret_cast<uint4*>(pdst + kPTile + g) = dk;
                if (j < P.S) *reinterpret_cast<uint4*>(ds_row + qc0 + e) = dk;
            }
            fence_proxy_async();
            mbar_arrive(p_full(x));
        }
        // ---------------- the accumulated key and value gradients of this tile
        mbar_wait(acc_done, 0, P.status, failed, 47);
        tc_fence_after();
        {
            const bool row_live = j < P.S;
            float* ok = P.dXK + ((int64_t)u * P.S + (row_live ? j : 0)) * kD + part * 32;
            float* ov = P.dXV + ((int64_t)u * P.S + (row_live ? j : 0)) * kD + part * 32;
#pragma unroll 1
            for (int mat = 0; mat < 2; ++mat) {
                uint32_t a[32];
                tmem_ld32(lane_base + (mat ? 384 : 256) + part * 32, a);     // (the whole warp, whatever its rows)
                tmem_ld_wait();
                if (row_live) {
                    float4* dst = reinterpret_cast<float4*>(mat ? ok : ov);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float4 cur = dst[e];
                        cur.x += __uint_as_float(a[4 * e]); cur.y += __uint_as_float(a[4 * e + 1]);
                        cur.z += __uint_as_float(a[4 * e + 2]); cur.w += __uint_as_float(a[4 * e + 3]);
                        dst[e] = cur;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace fused

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
    da_rows_kernel<<<U * (M / kDaRows), 256, 0, st>>>(p, dw, dab, dat, wb, L.Sp);
    if (!launched()) return -1;
    ++n;

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
    const Tensor4 t_xpad{xpad, {256, (uint64_t)L.Sp2, (uint64_t)U, 1}, {512, (uint64_t)L.Sp2 * 512, (uint64_t)U * L.Sp2 * 512}};
    const Tensor4 t_q = of_view(p.q, p.b, H, batch), t_do = of_view(p.d_o, p.b, H, batch);
    const int s_tiles = (S + 127) / 128;
    int n = 0;
    // blocks of queries: the buffer of dS^T (the former P and dS buffers together) holds 2 * QB queries
    const int QBf = 2 * L.QB;
    if (L.dsb <= L.pb || L.total - L.pb < (size_t)U * QBf * L.Sp * 2) return -1;   // the two regions follow each other
    __nv_bfloat16* dst_t = pb;                               // [unit][key][query of the block]
    static bool attr_set[64] = {};
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
        if (!attr_set[dev]) {
            if (cudaFuncSetAttribute(fused::attn_bwd_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, fused::kSmem) != cudaSuccess) return -1;
            attr_set[dev] = true;
        }
    }
    for (int q0 = 0; q0 < p.b; q0 += QBf) {
        const int qb = std::min(QBf, p.b - q0), q_tiles = (qb + 127) / 128;
        const int Sv = std::min(S, p.c + q0 + qb);          // keys any query of the block can see
        const int sv_tiles = (Sv + 127) / 128;
        {   // keys' side, fused: dX_V += P^T dO, dX_K += dS^T Q, and dS^T for the queries' side
            fused::Params F{};
            gemm::Operand ox, oq, od;
            if (!operand(ox, t_xpad, false) || !operand(oq, t_q, true) || !operand(od, t_do, true)) return -1;
            F.map_x = ox.map; F.map_q = oq.map; F.map_do = od.map;
            F.lse = p.lse + q0; F.lse_z = p.lse_stride;
            F.delta = p.delta + q0; F.delta_z = p.b;
            F.ds_t = dst_t; F.ds_z = (int64_t)L.Sp * QBf; F.ds_row = QBf;
            F.dXK = p.dXK; F.dXV = p.dXV;
            F.heads = H; F.S = S; F.c = p.c; F.pad = pad;
            F.q0 = q0; F.qb = qb; F.b = p.b;
            F.scale = p.scale; F.scale2 = p.scale * 1.4426950408889634f;
            F.status = reinterpret_cast<int*>(h->ws + h->off_status);
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3(sv_tiles, U);
            cfg.blockDim = dim3(fused::kThreads);
            cfg.dynamicSmemBytes = fused::kSmem;
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, fused::attn_bwd_kv_kernel, F) != cudaSuccess) {
                cudaGetLastError();
                return -1;
            }
            ++n;
        }
        {   // queries' side: dQ = dS X_K, with dS read as stored (keys along rows)
            gemm::Params G = base_params(h);
            const Tensor4 t_dst{dst_t, {(uint64_t)qb, (uint64_t)Sv, (uint64_t)U, 1}, {(uint64_t)QBf * 2, (uint64_t)L.Sp * QBf * 2, (uint64_t)U * L.Sp * QBf * 2}};
            if (!operand(G.A, t_dst, true) || !operand(G.B, t_xpad, true)) return -1;
            G.z_inner = H;
            G.A.c[0].tm = 128; G.A.c[1].si = 64; G.A.c[2].zi = 1; G.A.c[2].zo = H;
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
