// A batched bf16 GEMM on the 5th-generation tensor cores for the contractions of the backward pass:
//   D[z][m][n] (+)= alpha * sum_k A[m][k] * B[n][k]
// Operands come in through the tensor copy engine (128-byte swizzle) with tensor maps built by the
// caller, so "A[m][k]" is whatever the caller's map and coordinate rule make of it: either operand
// may be K-major (rows of K elements) or MN-major (rows of M/N elements, one row per k), and the
// coordinates of the box of K step s, output tile (tm, tn) and batch z are affine in
// (tm, tn % n_inner, tn / n_inner, s % s_inner, s / s_inner, z % z_inner, z / z_inner). That is enough for plain batched
// GEMMs, for sums over several units (the weight gradient), for row-shifted windows of one tensor
// (a convolution tap = a row offset; loads may start at negative rows and read zeros there) and for
// maps with overlapping strides (an im2col view that is never materialised).
// One CTA = one 128 x 128 output tile: one lane feeds a 3-stage ring (32 KB per stage), one lane issues
// four K=16 MMAs per stage into 128 TMEM columns, eight warps write the tile out (two per 32 rows).
// Two CTAs fit an SM, so one tile's epilogue overlaps the other's main loop.
#pragma once
#include <cuda.h>

#include <cstdint>

#include "tc_common.cuh"

namespace lococo {
namespace gemm {

using namespace tc;

struct Coord {      // one box coordinate = c0 + tm*TM + tni*(TN % n_inner) + tno*(TN / n_inner) + si*(s % s_inner) + so*(s / s_inner)
                    //                      + zi*(Z % z_inner) + zo*(Z / z_inner)
    int c0, tm, tni, tno, si, so, zi, zo;
};
struct Operand {
    CUtensorMap map;   // K-major: box {64 k, 128 rows}; MN-major: box {64 m/n, 64 k}, loaded at x and x + 64
    Coord c[4];
    int mn_major;
    int pad[3];
};
// kPairBF16: TWO products per tile, acc = A B^T and acc2 = A2 B2^T (same coordinates rule, second accumulator);
//            out  = p = exp2(acc * scale2 - rowvec[row] * log2 e) where column < causal_c + row + 1, else 0 (bf16)
//            out2 = p * (acc2 - rowvec2[row]) * alpha under the same mask (p in fp32: not rounded in between)
enum Mode { kStoreF32 = 0, kAtomicF32 = 1, kStoreBF16 = 2, kAddF32 = 3, kPairBF16 = 4 };
struct alignas(64) Params {
    Operand A, B;
    Operand A2, B2;              // second product of kPairBF16
    int n_inner, s_inner, z_inner;   // decomposition of the N tile index, of the K step index and of the batch index
    int steps, splits;           // K steps (64 wide) in total; CTAs that share them (blockIdx.z = z * splits + split)
    void* out;
    int64_t out_zi, out_zo, out_m;   // element strides of batch % z_inner, batch / z_inner and of a row
    int out_n_inner;             // column n lands at (n % out_n_inner) * out_n_in + (n / out_n_inner) * out_n_out
    int64_t out_n_in, out_n_out;
    int M, N;                    // valid rows and columns
    int mode;
    float alpha;
    int* status;
    // causal structure (rows = queries, columns = keys; row r sees columns < causal_c + r + 1)
    int causal_tiles;            // 1: output tiles entirely beyond the limit skip their K loop (and come out as zeros)
    int causal_c;
    int k_lo_on, k_lo_c0;        // K loop starts at step max(0, (tm * 128 + k_lo_c0) / 64)
    int k_hi_on, k_hi_c0;        // K loop ends before step (tm * 128 + k_hi_c0 + 63) / 64
    const float* rowvec;         // per (batch, row) values of kPairBF16
    int64_t rowvec_z;
    float scale2;
    void* out2;                  // kPairBF16
    const float* rowvec2;
    int64_t rowvec2_z;
};

constexpr int kThreads = 320;                      // 8 epilogue warps, the MMA-issue warp, the producer warp
constexpr int kStages = 3;
constexpr uint32_t kOperandBytes = 16384;
constexpr uint32_t kStageBytes2 = 2 * kOperandBytes;
constexpr uint32_t kSmem = kStages * kStageBytes2 + 1024 + 128;

__device__ __forceinline__ int coord_of(const Coord& c, const Params& P, int tm, int tn, int s, int z) {
    return c.c0 + c.tm * tm + c.tni * (tn % P.n_inner) + c.tno * (tn / P.n_inner) + c.si * (s % P.s_inner) + c.so * (s / P.s_inner) +
           c.zi * (z % P.z_inner) + c.zo * (z / P.z_inner);
}

__global__ void __launch_bounds__(kThreads, 2) gemm_kernel(const __grid_constant__ Params P) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes2);
    volatile int* failed = reinterpret_cast<volatile int*>(bars + 2 * kStages + 1);
    const uint32_t ring = smem_u32(smem), bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kStages, bar_acc = bar_empty + 8 * kStages;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int tm = blockIdx.x, tn = blockIdx.y;
    const int z = blockIdx.z / P.splits, split = blockIdx.z % P.splits;
    const int per = (P.steps + P.splits - 1) / P.splits;
    int s_begin = split * per, s_end = min(P.steps, s_begin + per);
    if (P.k_lo_on) s_begin = max(s_begin, max(0, tm * 128 + P.k_lo_c0) / 64);
    if (P.k_hi_on) s_end = min(s_end, max(0, tm * 128 + P.k_hi_c0 + 63) / 64);
    if (P.causal_tiles && tn * 128 >= P.causal_c + tm * 128 + 128) s_end = s_begin;
    if (s_end < s_begin) s_end = s_begin;
    const int passes = P.mode == kPairBF16 ? 2 : 1;

    if (tid == 256) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc, 1);
        *failed = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
    // launched as a programmatic dependent: the set-up above overlaps the previous kernel's tail, and
    // nothing global is touched before that kernel's results are complete and visible
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (tid == 288) {
        // ---- producer
        int g = 0;
        for (int pass = 0; pass < passes; ++pass)
        for (int s = s_begin; s < s_end; ++s, ++g) {
            const int st = g % kStages;
            if (g >= kStages) mbar_wait(bar_empty + 8 * st, ((g / kStages) - 1) & 1, P.status, failed, 30);
            mbar_expect_tx(bar_full + 8 * st, kStageBytes2);
            const uint32_t dst = ring + st * kStageBytes2;
#pragma unroll
            for (int op = 0; op < 2; ++op) {
                const Operand& O = pass ? (op ? P.B2 : P.A2) : (op ? P.B : P.A);
                const uint32_t d = dst + op * kOperandBytes;
                const int x = coord_of(O.c[0], P, tm, tn, s, z), y = coord_of(O.c[1], P, tm, tn, s, z);
                const int c2 = coord_of(O.c[2], P, tm, tn, s, z), c3 = coord_of(O.c[3], P, tm, tn, s, z);
                if (O.mn_major) {
                    tma_load_4d(d, &O.map, x, y, c2, c3, bar_full + 8 * st);
                    tma_load_4d(d + kOperandBytes / 2, &O.map, x + 64, y, c2, c3, bar_full + 8 * st);
                } else {
                    tma_load_4d(d, &O.map, x, y, c2, c3, bar_full + 8 * st);
                }
            }
        }
    } else if (tid == 256) {
        // ---- MMA issuer
        int g = 0;
        for (int pass = 0; pass < passes; ++pass)
        for (int s = s_begin; s < s_end; ++s, ++g) {
            const Operand& OA = pass ? P.A2 : P.A;
            const Operand& OB = pass ? P.B2 : P.B;
            const uint32_t idesc = instr_desc_bf16(128, OA.mn_major != 0, OB.mn_major != 0);
            const int st = g % kStages;
            mbar_wait(bar_full + 8 * st, (g / kStages) & 1, P.status, failed, 31);
            tc_fence_after();
            const uint32_t a_addr = ring + st * kStageBytes2, b_addr = a_addr + kOperandBytes;
            // K-major: 32 bytes per 16-element step inside the 128-byte row, 8-row groups 1024 bytes apart.
            // MN-major: 16 k rows (two 8-row groups) per step, the two 64-wide halves 8 KB apart.
            const uint64_t a0 = OA.mn_major ? smem_desc_sw128(a_addr, kOperandBytes / 2, 1024) : smem_desc_sw128(a_addr, 16, 1024);
            const uint64_t b0 = OB.mn_major ? smem_desc_sw128(b_addr, kOperandBytes / 2, 1024) : smem_desc_sw128(b_addr, 16, 1024);
            const uint32_t a_step = OA.mn_major ? 2048u >> 4 : 32u >> 4, b_step = OB.mn_major ? 2048u >> 4 : 32u >> 4;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_ss(tmem + pass * 128, a0 + kk * a_step, b0 + kk * b_step, idesc, (s != s_begin || kk != 0));
            umma_commit(bar_empty + 8 * st);
        }
        umma_commit(bar_acc);
    }
    if (warp < 8) {
        // ---- epilogue: thread = one row of the tile
        __syncwarp();
        const bool any = s_end > s_begin;
        if (any) {
            mbar_wait(bar_acc, 0, P.status, failed, 32);
            tc_fence_after();
        }
        // warp w reads TMEM lanes 32 * (w % 4) ..., i.e. those rows of the tile; warps 4-7 take columns 64-127
        const int row = tm * 128 + (tid & 127);
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const int c_begin = (tid >> 7) * 64;
        const int64_t base = (int64_t)(z % P.z_inner) * P.out_zi + (int64_t)(z / P.z_inner) * P.out_zo + (int64_t)row * P.out_m;
        const bool contiguous = P.out_n_in == 1 && P.out_n_inner % 32 == 0;
        if (P.mode == kPairBF16) {
            const float l2 = row < P.M ? P.rowvec[(int64_t)z * P.rowvec_z + row] * 1.4426950408889634f : 0.f;
            const float dl = row < P.M ? P.rowvec2[(int64_t)z * P.rowvec2_z + row] : 0.f;
            const int lim = min(P.N, P.causal_c + row + 1);       // columns this row sees
#pragma unroll 1
            for (int c0 = c_begin; c0 < c_begin + 64; c0 += 16) {
                uint32_t v[16], w[16];
                if (any) {
                    tmem_ld16(lane_addr + c0, v);
                    tmem_ld16(lane_addr + 128 + c0, w);
                    tmem_ld_wait();
                }
                const int n0 = tn * 128 + c0;
                if (row >= P.M || n0 >= P.N) continue;
                __nv_bfloat16* o1 = static_cast<__nv_bfloat16*>(P.out) + base + n0;
                __nv_bfloat16* o2 = static_cast<__nv_bfloat16*>(P.out2) + base + n0;
                uint32_t pk[8], dk[8];
#pragma unroll
                for (int e = 0; e < 16; e += 2) {
                    const bool on0 = any && n0 + e < lim, on1 = any && n0 + e + 1 < lim;
                    const float p0 = on0 ? exp2f(__uint_as_float(v[e]) * P.scale2 - l2) : 0.f;
                    const float p1 = on1 ? exp2f(__uint_as_float(v[e + 1]) * P.scale2 - l2) : 0.f;
                    const float d0 = on0 ? p0 * (__uint_as_float(w[e]) - dl) * P.alpha : 0.f;
                    const float d1 = on1 ? p1 * (__uint_as_float(w[e + 1]) - dl) * P.alpha : 0.f;
                    pk[e >> 1] = pack_bf16(p0, p1);
                    dk[e >> 1] = pack_bf16(d0, d1);
                }
                if (n0 + 16 <= P.N) {
                    *reinterpret_cast<uint4*>(o1) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *reinterpret_cast<uint4*>(o1 + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    *reinterpret_cast<uint4*>(o2) = make_uint4(dk[0], dk[1], dk[2], dk[3]);
                    *reinterpret_cast<uint4*>(o2 + 8) = make_uint4(dk[4], dk[5], dk[6], dk[7]);
                } else {
                    for (int e = 0; e < 16 && n0 + e < P.N; ++e) {
                        const uint32_t a = pk[e >> 1], d = dk[e >> 1];
                        reinterpret_cast<uint16_t*>(o1)[e] = (uint16_t)((e & 1) ? (a >> 16) : (a & 0xffffu));
                        reinterpret_cast<uint16_t*>(o2)[e] = (uint16_t)((e & 1) ? (d >> 16) : (d & 0xffffu));
                    }
                }
            }
        } else {
        const int mode = P.mode;
        const float alpha = P.alpha;
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_begin + 64; c0 += 32) {
            uint32_t v[32];
            if (any) {
                tmem_ld32(lane_addr + c0, v);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            const int n0 = tn * 128 + c0;
            if (row >= P.M || n0 >= P.N || (!any && mode != kStoreF32 && mode != kStoreBF16)) continue;
            const int64_t col0 = (int64_t)(n0 % P.out_n_inner) * P.out_n_in + (int64_t)(n0 / P.out_n_inner) * P.out_n_out;
            if (contiguous && n0 + 32 <= P.N) {
                if (mode == kStoreF32) {
                    float4* o = reinterpret_cast<float4*>(static_cast<float*>(P.out) + base + col0);
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        o[e >> 2] = make_float4(__uint_as_float(v[e]) * alpha, __uint_as_float(v[e + 1]) * alpha,
                                                __uint_as_float(v[e + 2]) * alpha, __uint_as_float(v[e + 3]) * alpha);
                } else if (mode == kAddF32) {
                    float4* o = reinterpret_cast<float4*>(static_cast<float*>(P.out) + base + col0);
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        float4 t = o[e >> 2];
                        t.x += __uint_as_float(v[e]) * alpha; t.y += __uint_as_float(v[e + 1]) * alpha;
                        t.z += __uint_as_float(v[e + 2]) * alpha; t.w += __uint_as_float(v[e + 3]) * alpha;
                        o[e >> 2] = t;
                    }
                } else if (mode == kStoreBF16) {
                    uint4* o = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + base + col0);
#pragma unroll
                    for (int e = 0; e < 32; e += 8)
                        o[e >> 3] = make_uint4(pack_bf16(__uint_as_float(v[e]) * alpha, __uint_as_float(v[e + 1]) * alpha),
                                               pack_bf16(__uint_as_float(v[e + 2]) * alpha, __uint_as_float(v[e + 3]) * alpha),
                                               pack_bf16(__uint_as_float(v[e + 4]) * alpha, __uint_as_float(v[e + 5]) * alpha),
                                               pack_bf16(__uint_as_float(v[e + 6]) * alpha, __uint_as_float(v[e + 7]) * alpha));
                } else {
                    float* o = static_cast<float*>(P.out) + base + col0;
#pragma unroll
                    for (int e = 0; e < 32; ++e) atomicAdd(o + e, __uint_as_float(v[e]) * alpha);
                }
            } else {
#pragma unroll 1
                for (int e = 0; e < 32; ++e) {
                    const int n = n0 + e;
                    if (n >= P.N) break;
                    const int64_t col = (int64_t)(n % P.out_n_inner) * P.out_n_in + (int64_t)(n / P.out_n_inner) * P.out_n_out;
                    const float x = __uint_as_float(v[e]) * alpha;
                    if (mode == kStoreF32) static_cast<float*>(P.out)[base + col] = x;
                    else if (mode == kAddF32) static_cast<float*>(P.out)[base + col] += x;
                    else if (mode == kStoreBF16) static_cast<__nv_bfloat16*>(P.out)[base + col] = __float2bfloat16_rn(x);
                    else atomicAdd(static_cast<float*>(P.out) + base + col, x);
                }
            }
        }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
    if (tid == 256) {
        for (int s = 0; s < 2 * kStages + 1; ++s) mbar_inval(bar_full + 8 * s);
    }
}

// ---- host side
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            sym = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

// bf16 tensor of rank 4: extents dims[0..3] (dims[0] innermost, contiguous), byte strides of dims 1..3.
// K-major operands take boxes of 64 x 128, MN-major operands boxes of 64 x 64.
inline bool make_map(CUtensorMap* map, const void* base, const uint64_t dims[4], const uint64_t strides[3], bool mn_major) {
    EncodeTiledFn fn = encode_tiled();
    if (!fn || (reinterpret_cast<uintptr_t>(base) & 15u)) return false;
    cuuint64_t d[4], s[3];
    for (int i = 0; i < 4; ++i) d[i] = dims[i] ? dims[i] : 1;
    for (int i = 0; i < 3; ++i) {
        s[i] = strides[i];
        if (s[i] == 0 || s[i] % 16 != 0 || s[i] >= ((cuuint64_t)1 << 40)) return false;
    }
    const cuuint32_t box[4] = {64, mn_major ? 64u : 128u, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), d, s, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch over (m_tiles, n_tiles, batch * splits). Returns false when the launch was refused.
inline bool launch(const Params& P, int m_tiles, int n_tiles, int batch, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess) return false;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(m_tiles, n_tiles, batch * P.splits);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, gemm_kernel, P) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}

}  // namespace gemm
}  // namespace lococo
