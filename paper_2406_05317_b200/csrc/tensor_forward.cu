// Tensor-core (tcgen05 / TMEM) kernels of the LoCoCo chunk step, bf16 storage, d = 128.
//
// compress_tc_kernel fuses Algorithm 2's Steps 4 and 5 for one tile of positions:
//   1. the [cache; chunk] key and value rows of the tile (plus a (k-1)/2 halo) are staged
//      once in shared memory by the tensor copy engine, as two 64-channel halves of 128-byte
//      rows in the 128-byte swizzle;
//   2. Eq. 6 runs as an implicit GEMM on the tensor cores: for every tap t,
//      D[slot, pos] += G_t[slot, ch] * Z[pos + t, ch]; a tap is a row offset into the
//      staged tile (the swizzle is a function of the shared-memory address, so an operand
//      may start at any row); the per-tap weight tiles stream from L2 through a ring fed by
//      bulk async copies;
//   3. the accumulator leaves TMEM once: bias, ReLU, the running row sum of Eq. 7, bf16
//      rounding, and the result is written back to shared memory as the A operand of
//   4. Eq. 4 / Eq. 5: U_K += R * X_K and U_V += R * X_V, which read the SAME staged tiles,
//      now contracted over positions (MN-major B operand);
// and the division by the row sum is applied after all tiles are summed (it commutes with the blend):
// by the CTA itself where it saw every position of its slots, by the CTA of a (unit, slot block) that
// arrives last at its store where the chunk loop lets the step merge its partial sets, and by
// finalize_parts_kernel after a stand-alone compress step.
#include <cuda.h>   // tensor map types only: the encoder is looked up at run time

#include <algorithm>
#include <type_traits>

#include "handle.h"
#include "tc_common.cuh"

namespace lococo {
namespace {

using namespace tc;

// The kernels of the chunk loop are launched so that they may start while the kernel before them in the
// stream drains (programmatic dependent launch): their CTAs take SMs as they fall free, let the kernel
// after them do the same, and wait for the earlier kernels' results only where they first need them —
// a step's attention CTAs before their cache tiles (which they process last), its compress CTAs before
// they stage cache rows or, if their tiles lie in the chunk, before they store their partial blends
// (the earlier finalize pass still reads that buffer). Everything before that point overlaps the tail
// of the previous step and its finalize pass. Without the launch attribute the wait is a no-op.
__device__ __forceinline__ void overlap_with_neighbours() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void wait_for_earlier_kernels() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}


constexpr int kSlots = 128;              // slots per CTA (MMA M)
constexpr int kD = 128;                  // head dimension
constexpr int kStageBytes = 32768;       // one tap x 128 channels x 128 slots, bf16
constexpr int kThreads = 384;            // twelve warps: see compress_body
constexpr int kMaxSmem = 232448 - 128;   // dynamic shared memory per CTA: 227 KB less the kernels' few static words
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColUK = 256, kColUV = 384;

struct TcCompressParams {
    CompressParams base;
    const __nv_bfloat16* gimage;  // [sets][slot blocks][k][halves][16][128][8]
    float* part_U;                // [units][slot blocks][parts][2][128 channels][128 slots]
    float* part_s;                // [units][slot blocks][parts][128]
    int part_stride;              // partial sets reserved per (unit, slot block): >= parts
    int direct;                   // 1 (only with parts == 1 and an output that is not the input cache): the CTA
                                  // normalises and writes the cache rows itself, no partials, no finalize pass
    float* R_store;               // optional [units][M][S]
    int* status;
    int merge;                    // 1 (parts > 1, output cache != input cache): the CTA that stores the last partial set of a
                                  // (unit, slot block) sums the sets and writes the cache rows itself, no finalize pass
    int* merge_count;             // [units][slot blocks][2]: CTAs arrived at their store, partial sets stored; the last CTA puts the zeros back
    int n_tile, tiles, parts, tiles_per_part, halves, stages, rows_pad, slot_blocks;
    int pair;                     // 1: generation-stage form, one CTA per TWO units that share a weight set (compress_pair_body)
    int pairs;                    // CTAs of that form
    // Tensor maps for staging the key and value tiles with the tensor copy engine (boxes of `rows` = n_tile + k - 1 token
    // rows x 64 channels, 128-byte swizzle), and for the tile (at most two) that holds both cache and chunk rows a pair of
    // maps with the box heights of its two parts. tile_maps == 0: every tile is staged by 16-byte async copies instead.
    int tile_maps;
    int seam_h1[2];               // cache rows (halo included) of a mixed tile; 0 = unused entry
    int out_maps;                 // 1: maps of the output cache (boxes of 128 slots x 64 channels) for the direct write
};
enum { kTmKCache = 0, kTmKChunk = 1, kTmVCache = 2, kTmVChunk = 3, kTmSeam = 4, kTmKOut = 12, kTmVOut = 13, kTileMaps = 14 };   // seam e: 4 + 4 e + {Kc, Kn, Vc, Vn}
struct alignas(64) TcTileMaps {
    CUtensorMap m[kTileMaps];
};

// G [sets][M][C][k] -> per (set, slot block, tap, 128-channel half) a 32 KB image of the
// K-major un-swizzled MMA operand: [16 channel groups][128 slots][8 channels].
__global__ void pack_image_kernel(const __nv_bfloat16* __restrict__ G, __nv_bfloat16* __restrict__ out, int sets, int M,
                                  int C, int k) {
    const int64_t total = (int64_t)sets * M * C * k;
    const int SB = M / kSlots, halves = C / 128;
    for (int64_t o = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int64_t r = o;
        const int e = r % 8; r /= 8;
        const int i = r % kSlots; r /= kSlots;
        const int q = r % 16; r /= 16;
        const int half = r % halves; r /= halves;
        const int t = r % k; r /= k;
        const int sb = r % SB;
        const int set = r / SB;
        const int slot = sb * kSlots + i, ch = half * 128 + q * 8 + e;
        out[o] = G[(((int64_t)set * M + slot) * C + ch) * k + t];
    }
}

// cache rows of slot block sb of unit u = (sum of the partial blends) / (sum of the partial row sums + eps), by the CTA
// (384 threads) that holds partial set `own` in its TMEM accumulators and its row sum in `own_s`; the other sets come
// from the workspace. The arithmetic is finalize_tile's, term for term, the sets added in their order. The threads are
// laid out as in the compress epilogues: a thread owns one slot (a warp 32 consecutive slots) and takes the eight
// (matrix, 32-channel chunk) pieces in turn with the two other warp groups; it ends up with 32 consecutive channels of
// its slot, 64 bytes of the slot-major cache row. The stored sets are channel-major and come in through the copy
// engine (a thread's own loads of them, 32 channels x 2 sets in flight around L1, left it waiting for an L2 round trip
// per piece: 6.5 us for two stored sets). A (matrix, 32-channel chunk) piece of a stored set is 16 KB of contiguous
// memory. Each of the three warp groups runs its pieces through a ring of three such buffers of its own: its first
// thread asks for the next pieces while the group adds up the ones that have arrived. `stage`: 3 x 3 x 16 KB of idle
// shared memory, 128-byte aligned (the host sets P.merge only where the ring and the tiles have room for it, which is
// every plan: at least two 32 KB stages and, where fewer than four fit, tiles of more than 99 KB); `bars`: nine
// barriers, already set up (one arrival each).
constexpr uint32_t kMergePiece = 32 * kSlots * 4;                 // bytes
constexpr uint32_t kMergeStage = 9 * kMergePiece;
__device__ __forceinline__ void merge_partials(const TcCompressParams& P, uint32_t tmem, int sb, int u, int own, float own_s,
                                               uint8_t* stage, uint32_t bars, volatile int* failed) {
    const CompressParams& p = P.base;
    const int n = u / p.heads, h = u % p.heads;
    const int warp = threadIdx.x >> 5;
    const int eg = warp >> 2, rl = (warp & 3) * 32 + (threadIdx.x & 31);
    const int slot = sb * kSlots + rl;
    const int64_t base = ((int64_t)u * P.slot_blocks + sb) * P.part_stride;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const bool leader = rl == 0;
    const int stored = P.parts - 1;                               // sets that come from memory
    const int n_pieces = (2 * (kD / 32) - eg + 2) / 3;            // pieces eg, eg + 3, ... below 8
    const int n_jobs = n_pieces * stored;
    const float* gbuf = reinterpret_cast<const float*>(stage + eg * 3 * kMergePiece);
    const uint32_t gbuf_a = smem_u32(gbuf), gbar = bars + eg * 24;
    // job j: stored set number (j % stored) of the group's piece number (j / stored), into buffer j % 3
    auto request = [&](int j) {
        const int piece = eg + 3 * (j / stored), k = j % stored;
        const int pt = k < own ? k : k + 1, mat = piece & 1, c0 = (piece >> 1) * 32;
        const uint32_t b = gbar + 8 * (j % 3);
        mbar_expect_tx(b, kMergePiece);
        bulk_load(gbuf_a + (j % 3) * kMergePiece, P.part_U + ((base + pt) * 2 + mat) * (int64_t)(kSlots * kD) + c0 * kSlots, kMergePiece, b);
    };
    if (leader) {
        // the sets were written by other CTAs' ordinary stores (seen through the acquire and the CTA barrier before this
        // call): ordered before the copy engine's reads of them
        asm volatile("fence.proxy.async;" ::: "memory");
        for (int j = 0; j < 3 && j < n_jobs; ++j) request(j);
    }
    float tot = 0.f;
    for (int pt = 0; pt < P.parts; ++pt) tot += pt == own ? own_s : __ldcg(P.part_s + (base + pt) * kSlots + rl);
    tot = slot < p.prot ? 1.f : tot + p.eps;   // a protected slot's row is e_i: denominator exactly 1
    const float inv = 1.f / tot;
    if (eg == 0) p.s[(int64_t)u * p.M + slot] = tot;
    int j = 0;
#pragma unroll 1
    for (int piece = eg; piece < 2 * (kD / 32); piece += 3) {
        const int mat = piece & 1, c0 = (piece >> 1) * 32;
        uint32_t mine[32];
        tmem_ld32(lane_addr + (mat ? kColUV : kColUK) + c0, mine);
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.f;
#pragma unroll 1
        for (int pt = 0; pt < P.parts; ++pt) {
            if (pt == own) {
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[e] += __uint_as_float(mine[e]);
                continue;
            }
            mbar_wait(gbar + 8 * (j % 3), (j / 3) & 1, P.status, failed, 14);
            const float* v = gbuf + (j % 3) * (kMergePiece / 4) + rl;
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] += v[e * kSlots];
            // the group is done with the buffer: its next use may be asked for
            asm volatile("bar.sync %0, 128;" ::"r"(3 + eg) : "memory");
            if (leader && j + 3 < n_jobs) request(j + 3);
            ++j;
        }
        const View& out = mat ? p.v_out : p.k_out;
        __nv_bfloat16* orow = unit_base_mut<__nv_bfloat16>(out, n, h) + (int64_t)slot * out.st + c0;
#pragma unroll
        for (int e = 0; e < 32; e += 8)
            *reinterpret_cast<uint4*>(orow + e) =
                make_uint4(pack_bf16(acc[e] * inv, acc[e + 1] * inv), pack_bf16(acc[e + 2] * inv, acc[e + 3] * inv),
                           pack_bf16(acc[e + 4] * inv, acc[e + 5] * inv), pack_bf16(acc[e + 6] * inv, acc[e + 7] * inv));
    }
}

// Work of one CTA of exactly 384 threads: tiles [part*tiles_per_part, ...) of slot block sb of unit u.
// Thread 128 issues the MMAs, thread 160 feeds the weight ring, every thread stages rows, and all
// twelve warps share the two epilogues: warp w owns accumulator rows (TMEM lanes) 32*(w%4)..+31
// and every third 32-column chunk, starting with chunk w/4.
// `tmem`: base of 512 TMEM columns the CTA owns. `cache_cg`: read cache rows around L1 (set when the
// cache was rewritten by other SMs earlier in the SAME kernel; L1 is coherent only across launches).
// kMerge: whether the kernel is one that may be asked to merge the partial sets itself (P.merge).
// `tmaps`: the tile maps in kernel parameter space, or nullptr (async-copy staging).
template <bool kMerge>
__device__ __forceinline__ void compress_body(const TcCompressParams& P, const TcTileMaps* tmaps, uint8_t* smem_raw, uint32_t tmem,
                                              bool cache_cg, int part, int sb, int u) {
    const CompressParams& p = P.base;
    // the tiles are 128-byte swizzled (a function of the shared-memory address): everything starts on a 1024-byte boundary
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int nthr16 = blockDim.x / 16;
    const int n = u / p.heads, h = u % p.heads;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int eg = warp >> 2;                          // epilogue group: which column chunks
    const int rl = (warp & 3) * 32 + (tid & 31);       // accumulator row = slot within the block
    const int n_tile = P.n_tile, pad = (p.k - 1) / 2, rows = n_tile + p.k - 1;
    const int NS = P.stages;
    const uint32_t half_z = (uint32_t)P.rows_pad * 128u;      // one 64-channel half of a tile: rows_pad rows of 128 bytes
    // does this CTA read cache rows (or write the cache itself)? then the earlier kernels come first
    const bool touches_cache = P.direct || part * P.tiles_per_part * n_tile - pad < p.xk.c;

    uint8_t* ring_ptr = smem;
    uint8_t* zk_ptr = ring_ptr + (size_t)NS * kStageBytes;
    uint8_t* zv_ptr = zk_ptr + 2 * half_z;
    uint64_t* bars = reinterpret_cast<uint64_t*>(zv_ptr + 2 * half_z);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * NS + 4);
    volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const uint32_t ring = smem_u32(ring_ptr), zk = smem_u32(zk_ptr), zv = smem_u32(zv_ptr);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * NS;
    const uint32_t bar_acc = bar_empty + 8 * NS, bar_blend = bar_acc + 8;
    const uint32_t bar_k = bar_blend + 8, bar_v = bar_k + 8;     // key tile, value tile staged

    if (warp == 4) {
        // every barrier here has one arrival per phase; a lane sets up one of them
        const int lane = tid & 31;
        if (lane < 2 * NS + 4) mbar_init(bar_full + 8 * lane, 1);
        if (lane == 0) *failed = 0;
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const int set = p.weights_per_head ? h : 0;
    const __nv_bfloat16* gimg =
        P.gimage + ((int64_t)set * P.slot_blocks + sb) * (int64_t)p.k * P.halves * (kStageBytes / 2);
    const uint32_t idesc_conv = instr_desc_bf16(n_tile, false, false);
    const uint32_t idesc_blend = instr_desc_bf16(kD, false, true);
    const int slot = sb * kSlots + rl;
    float bias_i = 0.f;
    if (p.bias) bias_i = p.bias[(p.weights_per_head ? h * p.M : 0) + slot];
    const __nv_bfloat16* safe = unit_base<__nv_bfloat16>(p.xk.chunk, n, h);

    float ssum = 0.f;
    uint32_t g = 0;  // ring stages used so far, over all tiles of this CTA
    const int tile_begin = part * P.tiles_per_part;
    const int tile_end = min(P.tiles, tile_begin + P.tiles_per_part);
    int tile_it = 0;
#pragma unroll 1
    for (int tile = tile_begin; tile < tile_end; ++tile, ++tile_it) {
        const int j0 = tile * n_tile;
        // columns of this tile that hold positions below S, as a multiple of 16: the last tile's MMAs are that narrow
        const int n_use = min(n_tile, (p.S - j0 + 15) & ~15);
        // The weight producer (one thread of warp 5) runs ahead of everything else: a tile's
        // first ring stages need no wait, the ring being drained at every tile boundary.
        const int total = p.k * P.halves;
        auto load_stage = [&](uint32_t gg, int it) {
            const uint32_t s = gg % NS;
            if (gg >= (uint32_t)NS) mbar_wait(bar_empty + 8 * s, ((gg / NS) - 1) & 1, P.status, failed, 1);
            mbar_expect_tx(bar_full + 8 * s, kStageBytes);
            bulk_load(ring + s * kStageBytes, gimg + (int64_t)it * (kStageBytes / 2), kStageBytes, bar_full + 8 * s);
        };
        const int npro = min(NS, total);
        if (tid == 160) {
            for (int i = 0; i < npro; ++i) load_stage(g + i, i);
        }
        // ---- 1. stage the key and value rows j0-pad .. j0+n_tile+pad-1 (zeros outside [0,S)) as two 64-channel halves
        // of 128-byte rows in the 128-byte swizzle. A tap is a row offset into the tile: the swizzle is a function of the
        // shared-memory address, so an operand may start at any row.
        // By the tensor copy engine where the tile's rows are one box of the cache or of the chunk, or (the tile that
        // holds the seam) one box of each with heights the host prepared; rows outside a tensor arrive as zeros.
        const int j_first = j0 - pad;
        const int h1 = p.xk.c > 0 ? max(0, min(rows, p.xk.c - j_first)) : 0;     // rows from the cache at the head of the tile
        int seam = -1;
        if (h1 > 0 && h1 < rows) seam = h1 == P.seam_h1[0] ? 0 : (h1 == P.seam_h1[1] ? 1 : -1);
        const bool by_engine = tmaps != nullptr && P.tile_maps && !cache_cg && (h1 == 0 || h1 == rows || seam >= 0);
        // one (matrix, source) box: both 64-channel halves
        auto engine_rows = [&](int map, int y, int dst_row, uint32_t dst, uint32_t bar) {
            tma_load_4d(dst + dst_row * 128, &tmaps->m[map], 0, y, h, n, bar);
            tma_load_4d(dst + half_z + dst_row * 128, &tmaps->m[map], 64, y, h, n, bar);
        };
        // `which` 0 keys, 1 values; `rows_of`: 0 all rows, 1 only rows outside the cache, 2 only cache rows
        auto engine_tile = [&](int which, uint32_t dst, uint32_t bar, int rows_of) {
            if (rows_of != 2) mbar_expect_tx(bar, (uint32_t)rows * 256u);
            if (h1 == rows) {
                if (rows_of != 1) engine_rows(kTmKCache + 2 * which, j_first, 0, dst, bar);
            } else if (h1 == 0) {
                if (rows_of != 2) engine_rows(kTmKChunk + 2 * which, j_first - p.xk.c, 0, dst, bar);
            } else {
                if (rows_of != 1) engine_rows(kTmSeam + 4 * seam + 2 * which, j_first, 0, dst, bar);
                if (rows_of != 2) engine_rows(kTmSeam + 4 * seam + 2 * which + 1, 0, h1, dst, bar);
            }
        };
        // the same tile by 16-byte async copies: each thread owns one 16-byte piece of a row (q) and every
        // (threads/16)-th row
        auto stage_tile = [&](const CatView& xv_, uint32_t dst, int first, int step, int rows_of = 0) {
            const int q = first & 15;
            const __nv_bfloat16* cbase = unit_base<__nv_bfloat16>(xv_.cache, n, h) + q * 8;
            const __nv_bfloat16* kbase = unit_base<__nv_bfloat16>(xv_.chunk, n, h) + q * 8;
            const uint32_t d0 = dst + (uint32_t)(q >> 3) * half_z;
            for (int r = first >> 4; r < rows; r += step) {
                const int j = j_first + r;
                const bool valid = j >= 0 && j < p.S;
                const bool in_cache = valid && j < xv_.c;
                if ((rows_of == 1 && in_cache) || (rows_of == 2 && !in_cache)) continue;
                const __nv_bfloat16* src = !valid ? safe : (in_cache ? cbase + (int64_t)j * xv_.cache.st
                                                                     : kbase + (int64_t)(j - xv_.c) * xv_.chunk.st);
                const uint32_t d = d0 + (uint32_t)r * 128u + (uint32_t)(((q & 7) ^ (r & 7)) << 4);
                if (in_cache && cache_cg) cp_async16_cg(d, src, 16u);
                else cp_async16(d, src, valid ? 16u : 0u);
            }
        };
        // the value tile is a conv input only when c_in = 2d; otherwise the blends alone need it
        if (by_engine) {
            // chunk rows (and the weight ring's first stages) before the wait for the previous step, cache rows after
            if (tid == 192) {
                engine_tile(0, zk, bar_k, touches_cache ? 1 : 0);
                engine_tile(1, zv, bar_v, touches_cache ? 1 : 0);
            }
            if (touches_cache) {
                wait_for_earlier_kernels();
                if (tid == 192) {
                    engine_tile(0, zk, bar_k, 2);
                    engine_tile(1, zv, bar_v, 2);
                }
            }
        } else {
            if (touches_cache) {
                stage_tile(p.xk, zk, tid, nthr16, 1);
                if (P.halves == 2) stage_tile(p.xv, zv, tid, nthr16, 1);
                wait_for_earlier_kernels();
                stage_tile(p.xk, zk, tid, nthr16, 2);
                if (P.halves == 2) stage_tile(p.xv, zv, tid, nthr16, 2);
            } else {
                stage_tile(p.xk, zk, tid, nthr16);
                if (P.halves == 2) stage_tile(p.xv, zv, tid, nthr16);
            }
            cp_async_wait_all();
            fence_proxy_async();
            __syncthreads();
            if (tid == 192) {
                mbar_arrive(bar_k);
                if (P.halves == 2) mbar_arrive(bar_v);
            }
        }

        // ---- 2. Eq. 6 as an implicit GEMM: one ring stage per (tap, 128-channel half).
        // Producer and MMA issuer are different threads, so the tensor pipe always has
        // several stages of MMAs queued while the next weight copies are in flight.
        if (tid == 160) {
            for (int it = npro; it < total; ++it) load_stage(g + it, it);
        } else if (tid == 128) {
            const uint64_t a0 = smem_desc(ring, 2048, 128);
            const uint64_t bk0 = smem_desc_sw128(zk, 16, 1024), bv0 = smem_desc_sw128(zv, 16, 1024);
            const uint32_t hstep = half_z >> 4;      // second 64-channel half of a tile
            const uint32_t idesc_tile = n_use == n_tile ? idesc_conv : instr_desc_bf16(n_use, false, false);
            mbar_wait(bar_k, tile_it & 1, P.status, failed, 5);
            if (P.halves == 2) mbar_wait(bar_v, tile_it & 1, P.status, failed, 6);
            // stage index and phase, tap and channel half are tracked incrementally: no division here
            uint32_t st = g % NS, ph = (g / NS) & 1, tap = 0, half = 0;
            for (int it = 0; it < total; ++it) {
                mbar_wait(bar_full + 8 * st, ph, P.status, failed, 2);
                tc_fence_after();
                const uint64_t ad = a0 + st * (uint32_t)(kStageBytes >> 4);
                const uint64_t bd = (half == 0 ? bk0 : bv0) + tap * 8u;   // tap t = row offset t (128 bytes per row)
                // 16 channels per step: 32 bytes inside the 128-byte row, then the tile's second half
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ss(tmem, ad + kk * 256u, bd + (uint32_t)(kk >> 2) * hstep + (uint32_t)(kk & 3) * 2u, idesc_tile, (it | kk) != 0);
                umma_commit(bar_empty + 8 * st);
                if (++half == (uint32_t)P.halves) { half = 0; ++tap; }
                if (++st == (uint32_t)NS) { st = 0; ph ^= 1; }
            }
            umma_commit(bar_acc);
        }
        g += total;

        // ---- 3. accumulator -> bias, ReLU, row sum (Eq. 7), bf16 -> A operand of the blends
        if (!by_engine && P.halves == 1 && (warp < 4 || warp >= 8)) {
            // (async-copy staging) the value tile, by the epilogue warps while the conv runs
            stage_tile(p.xv, zv, warp < 4 ? tid : tid - 128, 16);
            cp_async_wait_all();
        }
        __syncwarp();
        mbar_wait(bar_acc, tile_it & 1, P.status, failed, 3);
        tc_fence_after();
        {
            const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            float* rstore = P.R_store ? P.R_store + ((int64_t)u * p.M + slot) * p.S : nullptr;
            const bool keep = slot < p.prot;
            // (columns from n_use on were not written; they are read, as zeros, only by the copy of R for the backward pass)
            const int n_read = p.R16 ? n_tile : n_use;
#pragma unroll 1
            for (int c0 = eg * 32; c0 < n_read; c0 += 96) {
                uint32_t v[32];
                tmem_ld32(lane_addr + c0, v);
                tmem_ld_wait();
                const bool ragged = j0 + c0 + 32 > p.S;
                if (p.prot == 0 && !ragged && rstore == nullptr) {
                    // the common case, with as few instructions as it takes: round first, then clamp (rounding is monotonic
                    // and keeps zero, so max(round(x), 0) = round(max(x, 0))), two values per instruction
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int x = 0; x < 8; x += 2) {
                            const __nv_bfloat162 pr = __hmax2(__floats2bfloat162_rn(__uint_as_float(v[e + x]) + bias_i, __uint_as_float(v[e + x + 1]) + bias_i),
                                                              __floats2bfloat162_rn(0.f, 0.f));
                            pk[x >> 1] = *reinterpret_cast<const uint32_t*>(&pr);
                            ssum += __low2float(pr) + __high2float(pr);
                        }
                        *reinterpret_cast<uint4*>(ring_ptr + ((c0 + e) >> 3) * 2048 + rl * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                    continue;
                }
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    uint32_t pk[4];
#pragma unroll
                    for (int x = 0; x < 8; x += 2) {
                        const int ja = j0 + c0 + e + x;
                        float ra = fmaxf(__uint_as_float(v[e + x]) + bias_i, 0.f);
                        float rb = fmaxf(__uint_as_float(v[e + x + 1]) + bias_i, 0.f);
                        if (keep) { ra = ja == slot ? 1.f : 0.f; rb = ja + 1 == slot ? 1.f : 0.f; }   // unit row (Section 5.2)
                        if (ragged && ja >= p.S) ra = 0.f;
                        if (ragged && ja + 1 >= p.S) rb = 0.f;
                        const __nv_bfloat162 pr = __floats2bfloat162_rn(ra, rb);
                        pk[x >> 1] = *reinterpret_cast<const uint32_t*>(&pr);
                        const float fa = __low2float(pr), fb = __high2float(pr);
                        ssum += fa + fb;
                        if (rstore) {
                            if (ja < p.S) rstore[ja] = fa;
                            if (ja + 1 < p.S) rstore[ja + 1] = fb;
                        }
                    }
                    *reinterpret_cast<uint4*>(ring_ptr + ((c0 + e) >> 3) * 2048 + rl * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            fence_proxy_async();
        }
        tc_fence_before();
        __syncthreads();

        // ---- 4. Eq. 4, Eq. 5 (unnormalised): U_K += R X_K, U_V += R X_V from the staged tiles
        if (!by_engine && P.halves == 1 && tid == 192) mbar_arrive(bar_v);   // the barrier above covers the warps' copies
        if (tid == 128) {
            if (P.halves == 1) mbar_wait(bar_v, tile_it & 1, P.status, failed, 7);
            tc_fence_after();
#pragma unroll 1
            for (int kk = 0; kk < n_use / 16; ++kk) {
                // contraction over positions: 16 rows of the tiles per step (MN-major operands, the two 64-channel
                // blocks half a tile apart), starting `pad` rows in
                const uint64_t ad = smem_desc(ring + kk * 2 * 2048, 2048, 128);
                const uint32_t row0 = (uint32_t)(pad + kk * 16) * 128;
                const uint64_t bk = smem_desc_sw128(zk + row0, half_z, 1024);
                const uint64_t bv = smem_desc_sw128(zv + row0, half_z, 1024);
                const uint32_t acc = (tile_it | kk) != 0;
                umma_ss(tmem + kColUK, ad, bk, idesc_blend, acc);
                umma_ss(tmem + kColUV, ad, bv, idesc_blend, acc);
            }
            umma_commit(bar_blend);
        }
        // R as the blends read it (bf16, [position group][slot][8 positions]) also goes out row by row
        // when the backward pass asked for it: a slot's groups are consecutive 16-byte pieces of its row
        if (p.R16) {
            const int groups = n_tile / 8;
            __nv_bfloat16* r16 = static_cast<__nv_bfloat16*>(p.R16) + ((int64_t)u * p.M + sb * kSlots) * p.R16_stride + j0;
            for (int x = tid; x < kSlots * groups; x += blockDim.x) {
                const int sl = x / groups, gq = x % groups;
                if (j0 + gq * 8 < p.R16_stride)
                    *reinterpret_cast<uint4*>(r16 + (int64_t)sl * p.R16_stride + gq * 8) =
                        *reinterpret_cast<const uint4*>(ring_ptr + gq * 2048 + sl * 16);
            }
            __syncthreads();     // the ring is reused (row sums, next tile) once the blends are done
        }
        // the staged tiles and the ring are reused by the next tile only after the blends read them
        mbar_wait(bar_blend, tile_it & 1, P.status, failed, 4);
    }

    if (P.direct && tile_it > 0) {
        // ---- this CTA saw every position of its slots: Eq. 7 after Eq. 4-5 here, same arithmetic as finalize_tile
        tc_fence_after();
        float* sums = reinterpret_cast<float*>(ring_ptr);      // [3 groups][128 rows]; the ring is idle now
        sums[eg * kSlots + rl] = ssum;
        __syncthreads();
        const float tot = slot < p.prot ? 1.f : sums[rl] + sums[kSlots + rl] + sums[2 * kSlots + rl] + p.eps;
        const float inv = 1.f / tot;
        if (eg == 0) p.s[(int64_t)u * p.M + slot] = tot;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        // With maps of the output cache the rows leave through the copy engine: a thread (a slot) puts its 64-byte pieces
        // into four swizzled boxes of 128 slots x 64 channels in the idle ring, and one lane sends the boxes off. A warp
        // storing its 32 slots' pieces to memory itself pays for 32 separate segments per instruction.
        const bool by_store_engine = tmaps != nullptr && P.out_maps;
        uint8_t* boxes = ring_ptr + 2048;                      // [K | V][channels 0-63 | 64-127][128 slots][128 bytes]
#pragma unroll 1
        for (int piece = eg; piece < 2 * (kD / 32); piece += 3) {
            const int mat = piece & 1, c0 = (piece >> 1) * 32;
            uint32_t a[32];
            tmem_ld32(lane_addr + (mat ? kColUV : kColUK) + c0, a);
            tmem_ld_wait();
            uint4 o[4];
#pragma unroll
            for (int e = 0; e < 32; e += 8)
                o[e >> 3] = make_uint4(pack_bf16(__uint_as_float(a[e]) * inv, __uint_as_float(a[e + 1]) * inv),
                                       pack_bf16(__uint_as_float(a[e + 2]) * inv, __uint_as_float(a[e + 3]) * inv),
                                       pack_bf16(__uint_as_float(a[e + 4]) * inv, __uint_as_float(a[e + 5]) * inv),
                                       pack_bf16(__uint_as_float(a[e + 6]) * inv, __uint_as_float(a[e + 7]) * inv));
            if (by_store_engine) {
                uint8_t* row = boxes + (mat * 2 + (c0 >> 6)) * 16384 + rl * 128;
#pragma unroll
                for (int x = 0; x < 4; ++x) *reinterpret_cast<uint4*>(row + (((((c0 & 63) >> 3) + x) ^ (rl & 7)) << 4)) = o[x];
            } else {
                const View& out = mat ? p.v_out : p.k_out;
                __nv_bfloat16* orow = unit_base_mut<__nv_bfloat16>(out, n, h) + (int64_t)slot * out.st + c0;
#pragma unroll
                for (int x = 0; x < 4; ++x) *reinterpret_cast<uint4*>(orow + 8 * x) = o[x];
            }
        }
        if (by_store_engine) {
            fence_proxy_async();
            __syncthreads();
            if (tid == 0) {
#pragma unroll
                for (int x = 0; x < 4; ++x)
                    tma_store_4d(&tmaps->m[x < 2 ? kTmKOut : kTmVOut], smem_u32(boxes) + x * 16384, 64 * (x & 1), sb * kSlots, h, n);
                bulk_stores_read();
            }
        }
    } else
    // ---- partial blends and row sums of this CTA's tiles
    if (tile_it > 0) {
        if (!touches_cache) wait_for_earlier_kernels();      // the partial buffer may still be read by the last finalize pass
        tc_fence_after();
        float* sums = reinterpret_cast<float*>(ring_ptr);      // [3 groups][128 rows]; the ring is idle now
        sums[eg * kSlots + rl] = ssum;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const int64_t pidx = ((int64_t)u * P.slot_blocks + sb) * P.part_stride + part;
        // Where the step merges the sets itself (P.merge), the CTAs of a (unit, slot block) count in twice: on arrival
        // here, and once their set is stored. The one that arrives last keeps its set where it is (TMEM), waits for
        // the stored count of the others (CTAs that have arrived, so they are running and a few microseconds from
        // done; the wait is bounded all the same), and builds the cache rows. It puts both counts back to zero.
        int* counts = P.merge_count + 2 * ((int64_t)u * P.slot_blocks + sb);
        volatile int* is_last = reinterpret_cast<volatile int*>(ring_ptr + 4096);
        bool last = false;
        if (kMerge && P.merge) {
            if (tid == 0) *is_last = atomicAdd(counts, 1) == P.parts - 1;
            __syncthreads();
            last = *is_last != 0;
        }
        if (!last) {
            // stored channel-major ([channel][slot]) so that a warp's 32 lanes write 128 contiguous bytes;
            // the eight (matrix, 32-channel chunk) pieces go round the three groups. (Putting the set together in
            // shared memory first and sending it off as bulk copies, or as 16-byte stores by all threads, was 2-3 %
            // slower for a whole sequence: these stores leave straight from the accumulators and nothing waits for them.)
#pragma unroll 1
            for (int piece = eg; piece < 2 * (kD / 32); piece += 3) {
                const int mat = piece & 1, c0 = (piece >> 1) * 32;
                float* out = P.part_U + (pidx * 2 + mat) * (kSlots * kD) + rl;
                uint32_t a[32];
                tmem_ld32(lane_addr + (mat ? kColUV : kColUK) + c0, a);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) out[(c0 + e) * kSlots] = __uint_as_float(a[e]);
            }
            __syncthreads();
            if (tid < kSlots) P.part_s[pidx * kSlots + tid] = sums[tid] + sums[kSlots + tid] + sums[2 * kSlots + tid];
            if (kMerge && P.merge) {
                __threadfence();
                __syncthreads();
                if (tid == 0) atomicAdd(counts + 1, 1);
            }
        } else {
            if (tid == 0) {
                int seen = 0;
                const uint32_t limit = *failed ? 64u : (1u << 20);
                for (uint32_t i = 0; i < limit; ++i) {
                    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(counts + 1) : "memory");
                    if (seen >= P.parts - 1) break;
                    __nanosleep(32);
                }
                if (seen < P.parts - 1) {
                    *failed = 1;
                    atomicCAS(P.status, 0, 13);
                }
                counts[0] = 0;     // nobody touches the counts again before the next step
                counts[1] = 0;
            }
            // idle shared memory for the stored sets' pieces (past the row sums)
            uint8_t* stage = ring_ptr + 8192;
            const uint32_t mbars = smem_u32(ring_ptr + 2048);
            if (tid == 32) {
                for (int i = 0; i < 9; ++i) mbar_init(mbars + 8 * i, 1);
                fence_barrier_init();
            }
            __syncthreads();
            __threadfence();
            const float own_s = sums[rl] + sums[kSlots + rl] + sums[2 * kSlots + rl];
            merge_partials(P, tmem, sb, u, part, own_s, stage, mbars, failed);
        }
    }
    if (!kMerge) {
        // (a kernel whose CTA goes on to other work in this shared memory; a CTA that ends here leaves its barriers as they are)
        tc_fence_before();
        __syncthreads();
        if (warp == 4 && (tid & 31) < 2 * NS + 4) mbar_inval(bar_full + 8 * (tid & 31));
    }
}

// ------------------------------------------------------------------ generation stage (Section 3.3: segments of one token)
// With chunks of one (or a few) tokens S = c + b is barely larger than M: a compress step per unit is a single
// short position tile, and a CTA per unit streams the whole weight image (k stages of 32 KB) from L2 for about
// 130 positions, so with more units than SMs the step runs at what L2 delivers and not at the tensor pipe's rate.
// Here one CTA takes TWO units that use the same weight set: every weight stage feeds the MMAs of both (twice the
// MMA time per stage, half the weight traffic per unit). Conditions (checked on the host): M = 128, a full cache
// (c = M), c_in = d, one position tile (n_tile = S rounded up to 16), an output cache that is not the input cache.
//   TMEM: unit x owns columns 256x..256x+255: the conv accumulator D first (n_tile columns), and once D has been
//   turned into R in shared memory the two blend accumulators U_K, U_V (128 columns each) take its place.
//   Shared memory: [one region: the weight ring (4 stages) while the conv runs; afterwards R of both units and
//   the two value tiles of the cache rows, which only the blends need and which the tensor copy engine brings in
//   (128-byte swizzle, as the attention kernel's value tiles) while the accumulators are read out; at the end the
//   staging buffers of the cache write] [key tiles x2: rows -pad .. max(S+pad, n_tile)-1, un-swizzled].
//   The value blend runs on the tensor cores over the cache rows; the few chunk rows (positions c .. S-1) are added
//   on the CUDA cores from the same bf16 R (fp32 products and sums, as the MMA's).
// Units of pair `pair`: with one weight set for all heads, units 2*pair and 2*pair+1; with a set per head, the same
// head of sequences 2*i and 2*i+1 (pair = i*heads + head). The second unit may be missing (odd count).
__device__ __forceinline__ void pair_units(const CompressParams& p, int pair, int& u0, int& u1) {
    if (p.weights_per_head) {
        const int h = pair % p.heads, i = pair / p.heads, batch = p.units / p.heads;
        u0 = 2 * i * p.heads + h;
        u1 = 2 * i + 1 < batch ? u0 + p.heads : -1;
    } else {
        u0 = 2 * pair;
        u1 = u0 + 1 < p.units ? u0 + 1 : -1;
    }
}

constexpr int kPairStages = 4;
constexpr uint32_t kPairVTile = 32768;            // 128 cache rows x 128 channels, two 64-channel halves of 16 KB (128-byte swizzle)
constexpr uint32_t kPairOutRow = 272;             // bytes per row of a staged output tile: 256 + 16, so that 16-byte accesses of 8 rows miss each other's banks
constexpr uint32_t kPairOutTile = kSlots * kPairOutRow;

struct PairLayout {
    uint32_t rows_k, lbo_k, r_bytes, x_bytes, total;
};
__host__ __device__ inline PairLayout pair_layout(int S, int n_tile, int k) {
    const int pad = (k - 1) / 2;
    PairLayout L;
    // rows the conv reads for valid columns (S + k - 1) and rows the key blend reads (pad + n_tile), odd so that the 16
    // channel groups of a row fall into different banks
    L.rows_k = (uint32_t)(((S + k - 1 > pad + n_tile) ? S + k - 1 : pad + n_tile) | 1);
    L.lbo_k = L.rows_k * 16u;
    L.r_bytes = (uint32_t)(n_tile / 8) * 2048u;
    uint32_t x = kPairStages * (uint32_t)kStageBytes;
    if (x < 2u * L.r_bytes + 2u * kPairVTile) x = 2u * L.r_bytes + 2u * kPairVTile;
    if (x < 4u * kPairOutTile) x = 4u * kPairOutTile;
    L.x_bytes = x;
    L.total = 1024u + x + 2u * 16u * L.lbo_k + (2 * kPairStages + 3) * 8u + 16u + 2u * 3u * kSlots * 4u;
    return L;
}

// `vmap`: tensor map of the value cache ([batch, heads, c rows, 128] in boxes of 128 rows x 64 channels), in kernel
// parameter space.
__device__ __forceinline__ void compress_pair_body(const TcCompressParams& P, const CUtensorMap* vmap, const TcTileMaps* tmaps,
                                                   uint8_t* smem_raw, uint32_t tmem, int pair) {
    const CompressParams& p = P.base;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int eg = warp >> 2;                          // epilogue group: which column chunks
    const int rl = (warp & 3) * 32 + (tid & 31);       // accumulator row = slot
    const int n_tile = P.n_tile, pad = (p.k - 1) / 2;
    const PairLayout L = pair_layout(p.S, n_tile, p.k);
    const uint32_t lbo_k = L.lbo_k, r_bytes = L.r_bytes;
    int units[2];
    pair_units(p, pair, units[0], units[1]);
    const int nu = units[1] >= 0 ? 2 : 1;

    // the swizzle of the value tiles is a function of the shared-memory address: the region starts on a 1024-byte boundary
    uint8_t* x_ptr = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* zk_ptr = x_ptr + L.x_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(zk_ptr + 2 * 16 * lbo_k);
    volatile int* failed = reinterpret_cast<volatile int*>(bars + 2 * kPairStages + 3);
    float* sums = reinterpret_cast<float*>(const_cast<int*>(failed) + 4);          // [2 units][3 groups][128 rows]
    const uint32_t ring = smem_u32(x_ptr), zk = smem_u32(zk_ptr);
    const uint32_t vt = ring + 2 * r_bytes;                                         // value tiles, after R of both units
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kPairStages;
    const uint32_t bar_acc = bar_empty + 8 * kPairStages, bar_blend = bar_acc + 8, bar_v = bar_blend + 8;

    if (tid == 128) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_blend, 1);
        mbar_init(bar_v, 1);
        *failed = 0;
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const int h0 = units[0] % p.heads;
    const int set = p.weights_per_head ? h0 : 0;
    const __nv_bfloat16* gimg = P.gimage + (int64_t)set * p.k * (kStageBytes / 2);   // one slot block, one channel half
    const uint32_t idesc_conv = instr_desc_bf16(n_tile, false, false);
    const uint32_t idesc_blend = instr_desc_bf16(kD, false, true);
    const int slot = rl;
    float bias_i = 0.f;
    if (p.bias) bias_i = p.bias[(p.weights_per_head ? h0 * p.M : 0) + slot];
    const int total = p.k;

    auto load_stage = [&](int it) {
        const uint32_t s = it % kPairStages;
        if (it >= kPairStages) mbar_wait(bar_empty + 8 * s, ((it / kPairStages) - 1) & 1, P.status, failed, 31);
        mbar_expect_tx(bar_full + 8 * s, kStageBytes);
        bulk_load(ring + s * kStageBytes, gimg + (int64_t)it * (kStageBytes / 2), kStageBytes, bar_full + 8 * s);
    };
    if (tid == 160) {
        for (int i = 0; i < min(kPairStages, total); ++i) load_stage(i);
    }
    // ---- 1. stage the key rows: the tile of unit x holds positions -pad .. rows_k-pad-1 (zeros outside [0,S)).
    // Each thread owns one 8-channel group and every 24th row. `rows_of`: 1 only rows outside the cache (chunk rows and
    // zeros), 2 only cache rows.
    auto stage_keys = [&](int x, int rows_of) {
        const int u = units[x], n = u / p.heads, h = u % p.heads;
        const int q = tid & 15;
        const __nv_bfloat16* cbase = unit_base<__nv_bfloat16>(p.xk.cache, n, h) + q * 8;
        const __nv_bfloat16* kbase = unit_base<__nv_bfloat16>(p.xk.chunk, n, h) + q * 8;
        const uint32_t d0 = zk + x * 16 * lbo_k + q * lbo_k;
        for (int r = tid >> 4; r < (int)L.rows_k; r += kThreads / 16) {
            const int j = r - pad;
            const bool valid = j >= 0 && j < p.S;
            const bool in_cache = valid && j < p.xk.c;
            if ((rows_of == 1 && in_cache) || (rows_of == 2 && !in_cache)) continue;
            const __nv_bfloat16* src = !valid ? kbase : (in_cache ? cbase + (int64_t)j * p.xk.cache.st : kbase + (int64_t)(j - p.xk.c) * p.xk.chunk.st);
            cp_async16(d0 + r * 16, src, valid ? 16u : 0u);
        }
    };
    for (int x = 0; x < nu; ++x) stage_keys(x, 1);
    wait_for_earlier_kernels();          // the cache rows are the previous step's result
    for (int x = 0; x < nu; ++x) stage_keys(x, 2);
    cp_async_wait_all();
    fence_proxy_async();
    __syncthreads();

    // ---- 2. Eq. 6: every weight stage (one tap) feeds both units' accumulators
    if (tid == 160) {
        for (int it = kPairStages; it < total; ++it) load_stage(it);
    } else if (tid == 128) {
        const uint64_t a0 = smem_desc(ring, 2048, 128);
        const uint64_t b0 = smem_desc(zk, lbo_k, 128), b1 = smem_desc(zk + 16 * lbo_k, lbo_k, 128);
        const uint32_t bstep = (2 * lbo_k) >> 4;
        uint32_t st = 0, ph = 0;
        for (int it = 0; it < total; ++it) {
            mbar_wait(bar_full + 8 * st, ph, P.status, failed, 32);
            tc_fence_after();
            const uint64_t ad = a0 + st * (uint32_t)(kStageBytes >> 4);
            umma_ss_k8(tmem, ad, b0 + it, 256u, bstep, idesc_conv, it != 0);              // tap t = row offset t (16 bytes per row)
            if (nu == 2) umma_ss_k8(tmem + 256, ad, b1 + it, 256u, bstep, idesc_conv, it != 0);
            umma_commit(bar_empty + 8 * st);
            if (++st == (uint32_t)kPairStages) { st = 0; ph ^= 1; }
        }
        umma_commit(bar_acc);
    }
    mbar_wait(bar_acc, 0, P.status, failed, 33);
    tc_fence_after();
    // the ring is idle now: the value tiles of the cache rows (needed by the blends only) are requested here, through
    // the tensor copy engine, and arrive while the accumulators are read out
    if (tid == 160) {
        mbar_expect_tx(bar_v, (uint32_t)nu * kPairVTile);
        for (int x = 0; x < nu; ++x) {
            const int u = units[x], n = u / p.heads, h = u % p.heads;
            tma_load_4d(vt + x * kPairVTile, vmap, 0, 0, h, n, bar_v);
            tma_load_4d(vt + x * kPairVTile + kPairVTile / 2, vmap, 64, 0, h, n, bar_v);
        }
    }

    // ---- 3. accumulators -> bias, ReLU, row sums (Eq. 7), bf16 -> A operands of the blends (over the idle ring)
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const bool keep = slot < p.prot;
#pragma unroll 1                                  // (one copy of the code for both units: code that runs once costs its own fetch)
    for (int x = 0; x < nu; ++x) {
        {
            float ssum = 0.f;
            for (int c0 = eg * 32; c0 < n_tile; c0 += 96) {
                uint32_t v[32];
                tmem_ld32(lane_addr + x * 256 + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    if (c0 + e >= n_tile) break;          // n_tile is a multiple of 16, not of 32
                    uint32_t pk[4];
#pragma unroll
                    for (int y = 0; y < 8; y += 2) {
                        const int ja = c0 + e + y;
                        float ra = fmaxf(__uint_as_float(v[e + y]) + bias_i, 0.f);
                        float rb = fmaxf(__uint_as_float(v[e + y + 1]) + bias_i, 0.f);
                        if (keep) { ra = ja == slot ? 1.f : 0.f; rb = ja + 1 == slot ? 1.f : 0.f; }   // unit row (Section 5.2)
                        if (ja >= p.S) ra = 0.f;
                        if (ja + 1 >= p.S) rb = 0.f;
                        const __nv_bfloat162 pr = __floats2bfloat162_rn(ra, rb);
                        pk[y >> 1] = *reinterpret_cast<const uint32_t*>(&pr);
                        ssum += __low2float(pr) + __high2float(pr);
                    }
                    *reinterpret_cast<uint4*>(x_ptr + x * r_bytes + ((c0 + e) >> 3) * 2048 + rl * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            sums[(x * 3 + eg) * kSlots + rl] = ssum;
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();

    // ---- 4. Eq. 4, Eq. 5 (unnormalised) into the columns the conv accumulators occupied: keys over all positions
    // from the staged key tiles, values over the cache rows from the swizzled tiles
    if (tid == 128) {
        tc_fence_after();
        for (int x = 0; x < nu; ++x) {
            uint64_t ad = smem_desc(ring + x * r_bytes, 2048, 128);
            uint64_t bk = smem_desc(zk + x * 16 * lbo_k + (uint32_t)pad * 16, 128, lbo_k);
            for (int kk = 0; kk < n_tile / 16; ++kk) {
                umma_ss(tmem + x * 256, ad, bk, idesc_blend, kk != 0);
                ad += (2 * 2048) >> 4;      // 16 positions = two 8-position groups of R
                bk += (16 * 16) >> 4;       // 16 rows of the key tile
            }
        }
        mbar_wait(bar_v, 0, P.status, failed, 35);
        tc_fence_after();
        for (int x = 0; x < nu; ++x) {
            const uint64_t ad = smem_desc(ring + x * r_bytes, 2048, 128);
            const uint64_t bv = smem_desc_sw128(vt + x * kPairVTile, kPairVTile / 2, 1024);
            // 16 cache rows = two 8-row groups of 1024 bytes per step
            umma_ss_k8(tmem + x * 256 + 128, ad, bv, 256u, 128u, idesc_blend, 0);
        }
        umma_commit(bar_blend);
    }
    mbar_wait(bar_blend, 0, P.status, failed, 34);
    tc_fence_after();

    // ---- 5. Eq. 7 after Eq. 4-5: add the chunk rows' share of the value blend, divide by the row sum, and write the
    // cache rows. A thread owns a slot; the rows are staged in shared memory so that the stores to the cache are
    // whole 256-byte rows (a warp storing 32 rows' pieces directly pays for 32 separate segments per instruction).
    const int n_tail = p.S - p.xk.c;                     // chunk rows: positions c .. S-1 (<= 16 of them)
    const bool by_store_engine = tmaps != nullptr && P.out_maps;   // the cache rows leave as boxes through the copy engine
    float rtail[2][16];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        const uint8_t* rrow = x_ptr + x * r_bytes + rl * 16;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
            if (x < nu && p.xk.c + 8 * g < n_tile) w4 = *reinterpret_cast<const uint4*>(rrow + ((p.xk.c >> 3) + g) * 2048);
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&w4);
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const float2 f = __bfloat1622float2(h2[y]);
                rtail[x][8 * g + 2 * y] = f.x;
                rtail[x][8 * g + 2 * y + 1] = f.y;
            }
        }
    }
    __syncthreads();                                      // R has been read: its space now stages the output rows
#pragma unroll 1
    for (int x = 0; x < nu; ++x) {
        const int u = units[x], n = u / p.heads, h = u % p.heads;
        const float tot = slot < p.prot ? 1.f : sums[(x * 3) * kSlots + rl] + sums[(x * 3 + 1) * kSlots + rl] + sums[(x * 3 + 2) * kSlots + rl] + p.eps;
        const float inv = 1.f / tot;
        if (eg == 0) p.s[(int64_t)u * p.M + slot] = tot;
        const __nv_bfloat16* vn = unit_base<__nv_bfloat16>(p.xv.chunk, n, h);
#pragma unroll 1
        for (int piece = eg; piece < 2 * (kD / 32); piece += 3) {
            const int mat = piece & 1, c0 = (piece >> 1) * 32;
            uint32_t a[32];
            tmem_ld32(lane_addr + x * 256 + mat * 128 + c0, a);
            tmem_ld_wait();
            float acc[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] = __uint_as_float(a[e]);
            if (mat == 1) {
#pragma unroll
                for (int y = 0; y < 16; ++y) {
                    if (y >= n_tail) break;
                    const float w = x == 0 ? rtail[0][y] : rtail[1][y];
                    const uint4* row = reinterpret_cast<const uint4*>(vn + (int64_t)y * p.xv.chunk.st + c0);   // the same 64 bytes for the whole warp
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const uint4 v4 = row[g];
                        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v4);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 f = __bfloat1622float2(h2[e]);
                            acc[8 * g + 2 * e] = fmaf(w, f.x, acc[8 * g + 2 * e]);
                            acc[8 * g + 2 * e + 1] = fmaf(w, f.y, acc[8 * g + 2 * e + 1]);
                        }
                    }
                }
            }
            uint4 o[4];
#pragma unroll
            for (int e = 0; e < 32; e += 8)
                o[e >> 3] = make_uint4(pack_bf16(acc[e] * inv, acc[e + 1] * inv), pack_bf16(acc[e + 2] * inv, acc[e + 3] * inv),
                                       pack_bf16(acc[e + 4] * inv, acc[e + 5] * inv), pack_bf16(acc[e + 6] * inv, acc[e + 7] * inv));
            if (by_store_engine) {
                // swizzled boxes of 128 slots x 64 channels: [unit][K | V][channels 0-63 | 64-127]
                uint8_t* row = x_ptr + ((x * 2 + mat) * 2 + (c0 >> 6)) * 16384 + rl * 128;
#pragma unroll
                for (int y = 0; y < 4; ++y) *reinterpret_cast<uint4*>(row + (((((c0 & 63) >> 3) + y) ^ (rl & 7)) << 4)) = o[y];
            } else {
                uint8_t* orow = x_ptr + (x * 2 + mat) * kPairOutTile + rl * kPairOutRow + c0 * 2;
#pragma unroll
                for (int y = 0; y < 4; ++y) *reinterpret_cast<uint4*>(orow + 16 * y) = o[y];
            }
        }
    }
    if (by_store_engine) {
        // the copy engine takes the boxes to the cache
        fence_proxy_async();
        __syncthreads();
        if (tid == 0) {
            for (int x = 0; x < nu; ++x) {
                const int u = units[x], n = u / p.heads, h = u % p.heads;
#pragma unroll
                for (int y = 0; y < 4; ++y)
                    tma_store_4d(&tmaps->m[y < 2 ? kTmKOut : kTmVOut], smem_u32(x_ptr) + (x * 4 + y) * 16384, 64 * (y & 1), 0, h, n);
            }
            bulk_stores_read();
        }
    } else {
    __syncthreads();
#pragma unroll 1
    for (int x = 0; x < nu; ++x) {
        const int u = units[x], n = u / p.heads, h = u % p.heads;
#pragma unroll 1
        for (int mat = 0; mat < 2; ++mat) {
            const View& out = mat ? p.v_out : p.k_out;
            __nv_bfloat16* obase = unit_base_mut<__nv_bfloat16>(out, n, h);
            const uint8_t* tile = x_ptr + (x * 2 + mat) * kPairOutTile;
            for (int idx = tid; idx < kSlots * 16; idx += kThreads) {
                const int row = idx >> 4, piece16 = idx & 15;
                *reinterpret_cast<uint4*>(obase + (int64_t)row * out.st + piece16 * 8) =
                    *reinterpret_cast<const uint4*>(tile + row * kPairOutRow + piece16 * 16);
            }
        }
    }
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 128) {
        for (int s = 0; s < 2 * kPairStages + 3; ++s) mbar_inval(bar_full + 8 * s);
    }
}

// The CTA's TMEM (all 512 columns; one CTA per SM) is allocated around the work, not inside it.
__device__ __forceinline__ uint32_t cta_tmem_acquire(uint32_t* slot) {
    if (threadIdx.x < 32) {
        tmem_alloc(smem_u32(slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    return *reinterpret_cast<volatile uint32_t*>(slot);
}
__device__ __forceinline__ void cta_tmem_release(uint32_t tmem) {
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem, kTmemCols);
}

struct TcCompressLaunch {
    TcCompressParams c;
    TcTileMaps t;
};
__global__ void __launch_bounds__(kThreads, 1) compress_tc_kernel(const __grid_constant__ TcCompressLaunch P) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t tmem_slot;
    const uint32_t tmem = cta_tmem_acquire(&tmem_slot);
    compress_body<false>(P.c, &P.t, smem, tmem, false, blockIdx.x, blockIdx.y, blockIdx.z);
    cta_tmem_release(tmem);
}

// cache = (sum of partial blends) / (sum of partial row sums + eps)   (Eq. 7 after Eq. 4-5)
// One block per 32 slots x 32 channels: the partials are channel-major (read along slots),
// the cache is slot-major (written along channels); the tile is transposed in shared memory.
// Runs with at least 256 threads; threads beyond the first 256 only take part in the barriers.
// Partials are read around L1 (__ldcg): in the persistent kernel other SMs wrote them moments ago.
__device__ __forceinline__ void finalize_tile(const TcCompressParams& P, float (*tk)[33], float (*tv)[33], float* inv_s,
                                              int bx, int by, int u) {
    const CompressParams& p = P.base;
    const int n = u / p.heads, h = u % p.heads;
    const int i0 = bx * 32, c0 = by * 32;   // slot tile, channel tile
    const int sb = i0 / kSlots, il0 = i0 % kSlots;
    const int64_t base = ((int64_t)u * P.slot_blocks + sb) * P.part_stride;
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
    __syncthreads();                            // the tile buffers may still be read by the previous tile
    if (ty == 0) {
        float s = 0.f;
        for (int pt = 0; pt < P.parts; ++pt) s += __ldcg(P.part_s + (base + pt) * kSlots + il0 + tx);
        s = i0 + tx < p.prot ? 1.f : s + p.eps;   // a protected slot's row is e_i: denominator exactly 1
        inv_s[tx] = 1.f / s;
        if (c0 == 0) p.s[(int64_t)u * p.M + i0 + tx] = s;
    }
    if (ty < 8) {
        for (int cc = ty; cc < 32; cc += 8) {      // tx runs along slots: 128-byte coalesced reads
            float uk = 0.f, uv = 0.f;
            for (int pt = 0; pt < P.parts; ++pt) {
                uk += __ldcg(P.part_U + ((base + pt) * 2 + 0) * (kSlots * kD) + (c0 + cc) * kSlots + il0 + tx);
                uv += __ldcg(P.part_U + ((base + pt) * 2 + 1) * (kSlots * kD) + (c0 + cc) * kSlots + il0 + tx);
            }
            tk[cc][tx] = uk;
            tv[cc][tx] = uv;
        }
    }
    __syncthreads();
    if (ty < 8) {
        for (int ii = ty; ii < 32; ii += 8) {      // tx runs along channels: coalesced writes
            const float inv = inv_s[ii];
            const int64_t row = (int64_t)(i0 + ii);
            unit_base_mut<__nv_bfloat16>(p.k_out, n, h)[row * p.k_out.st + c0 + tx] = __float2bfloat16_rn(tk[tx][ii] * inv);
            unit_base_mut<__nv_bfloat16>(p.v_out, n, h)[row * p.v_out.st + c0 + tx] = __float2bfloat16_rn(tv[tx][ii] * inv);
        }
    }
}

__global__ void __launch_bounds__(256) finalize_parts_kernel(TcCompressParams P) {
    __shared__ float tk[32][33], tv[32][33], inv_s[32];
    overlap_with_neighbours();
    wait_for_earlier_kernels();
    finalize_tile(P, tk, tv, inv_s, blockIdx.x, blockIdx.y, blockIdx.z);
}

// ------------------------------------------------------------------ Eq. 1, chunk form
// One CTA = 128 queries of one unit, pipelined over 128-key tiles of [cache; chunk] with three
// kinds of warps that only meet at mbarriers:
//   loaders (3 warps)   one lane drives the tensor copy engine: Q once, then the K/V tiles, double-buffered;
//                       the warps copy by hand (cp.async) only the tile that straddles the end of a
//                       partly filled cache, or an operand whose strides the driver would not encode;
//   MMA issuer (1 lane) S_t = Q K_t^T into one of two TMEM buffers, then O += P_{t-1} V_{t-1},
//                       so the next tile's logits are computed while this tile's softmax runs;
//   softmax (8 warps)   two threads per query row (64 columns each): row maximum, P = exp2(s - m)
//                       in bf16 to shared memory (double-buffered MMA A operand), running row sum.
// O stays in TMEM for the whole CTA. The reference maximum m of a row is raised only when a
// tile's maximum exceeds it by more than 8 (in log2 units): P then reaches at most 2^8, which
// bf16 and the fp32 accumulator hold just as well, and the rescale of O (a TMEM round trip)
// becomes rare; all sums use the same m, so the result is the exact softmax.
constexpr int kAttnThreads = 384;                  // 8 softmax + 1 MMA-issue + 3 loader warps (384 x 168 registers fill the file)
constexpr int kAttnLoaderWarps = 3;
constexpr int kAttnLoaders = 32 * kAttnLoaderWarps;
constexpr uint32_t kHalfBytes = 16384;             // 128 rows x 64 channels: rows of 128 bytes, 128-byte swizzle
constexpr uint32_t kTileBytes = 2 * kHalfBytes;    // Q/K/V tiles: channels 0-63, then channels 64-127
constexpr uint32_t kPBytes = 32768;                // P tiles: [16 key groups][128 rows][8 keys], no swizzle
constexpr uint32_t kAttnSmem = 5 * kTileBytes + 2 * kPBytes + 256 * 4 + 128 + 1024;   // Q, K x2, V x2, P x2, exchange, barriers, alignment
constexpr uint32_t kAttnTmemCols = 512;            // S x2 (128 columns each), O (128)
constexpr float kRescaleThreshold = 8.f;

// Tensor maps of the five operands: [batch, heads, tokens, 128] bf16 views cut into boxes of 128 tokens x
// 64 channels. A map the driver would not encode (its bit in tma_mask clear) leaves that operand to the
// loader warps' 16-byte copies, which write the same swizzled tile.
enum { kMapQ = 0, kMapKChunk = 1, kMapVChunk = 2, kMapKCache = 3, kMapVCache = 4, kMaps = 5 };
struct alignas(64) TcAttnParams {
    CUtensorMap maps[kMaps];
    AttnParams base;
    int* status;
    unsigned tma_mask;
};

// Work of one CTA (exactly kAttnThreads threads): query tile qtile of unit u. `tmem`: as for
// compress_body. `maps`: P.maps where the copy engine can read them (kernel parameter space or global
// memory); `maps_fresh`: they were written to global memory after an earlier kernel used that address.
__device__ __forceinline__ void attention_body(const TcAttnParams& P, const CUtensorMap* maps, bool maps_fresh, uint8_t* smem_raw,
                                               uint32_t tmem, int qtile, int u) {
    const AttnParams& p = P.base;
    const int n = u / p.heads, h = u % p.heads;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r0 = qtile * 128;
    const int S = p.c + p.b;

    // the swizzle is a function of the shared-memory address: tiles start on 1024-byte boundaries
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* q_ptr = smem;
    uint8_t* k_ptr = q_ptr + kTileBytes;       // two buffers
    uint8_t* v_ptr = k_ptr + 2 * kTileBytes;   // two buffers
    uint8_t* p_ptr = v_ptr + 2 * kTileBytes;   // two buffers
    float* xchg = reinterpret_cast<float*>(p_ptr + 2 * kPBytes);      // [2 halves][128 rows]
    uint64_t* bars = reinterpret_cast<uint64_t*>(xchg + 256);
    volatile int* failed = reinterpret_cast<volatile int*>(bars + 13);
    const uint32_t qs = smem_u32(q_ptr), ks = smem_u32(k_ptr), vs = smem_u32(v_ptr), ps = smem_u32(p_ptr);
    const uint32_t bar0 = smem_u32(bars);
    // all indexed by b = tile & 1; the n-th use of a buffer completes phase n of its barriers
    auto k_full = [&](int b) { return bar0 + 8 * b; };          // loader -> MMA: K tile staged
    auto v_full = [&](int b) { return bar0 + 80 + 8 * b; };     // loader -> MMA: V tile staged
    auto s_full = [&](int b) { return bar0 + 16 + 8 * b; };     // MMA -> softmax: logits in TMEM
    auto s_free = [&](int b) { return bar0 + 32 + 8 * b; };     // softmax -> MMA: logits consumed
    auto p_full = [&](int b) { return bar0 + 48 + 8 * b; };     // softmax -> MMA: P written
    auto pv_done = [&](int b) { return bar0 + 64 + 8 * b; };    // MMA -> loader, softmax: K/V/P buffers free, O updated
    const uint32_t q_full = bar0 + 96;                          // loader -> MMA: Q tile staged
    constexpr int kMma = 256;                                   // lane 0 of warp 8
    constexpr int kLoad = 288;                                  // lane 0 of warp 9: issues the tensor copies

    if (warp == kMma / 32) {
        // a lane sets up one of the thirteen barriers: s_free and p_full (words 4-7) count the 256 softmax threads
        const int lane = tid & 31;
        if (lane < 13) mbar_init(bar0 + 8 * lane, lane >= 4 && lane < 8 ? 256 : 1);
        if (lane == 0) *failed = 0;
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const int last_row = min(r0 + 127, p.b - 1);
    const int ncols = p.c + last_row + 1;           // columns any query of this tile can see
    const int ntiles = (ncols + 127) / 128;
    // Key tiles are processed chunk first, cache last (the softmax does not care about the order): the tiles
    // that hold cache rows are the only ones that depend on the previous step's result.
    const int cache_tiles = min(ntiles, (p.c + 127) / 128);
    auto tile_of = [&](int jt) { const int a = jt + cache_tiles; return a >= ntiles ? a - ntiles : a; };

    if (warp >= 9) {
        // ---------------- loader: one lane drives the copy engine; the three warps together stage what
        // the engine cannot (an operand without a tensor map, the tile that straddles the end of the cache)
        const int lw = warp - 9;
        const bool elected = tid == kLoad;
        const unsigned mask = P.tma_mask;
        const __nv_bfloat16* safe = unit_base<__nv_bfloat16>(p.q, n, h);
        if (elected && maps_fresh) {
            for (int i = 0; i < kMaps; ++i)
                if ((mask >> i) & 1) tensormap_acquire(maps + i);
        }
        // one 128-row tile through the engine: both 64-channel halves, signalled on `bar` as bytes
        auto engine_tile = [&](uint32_t dst, uint32_t bar, int mi, int token) {
            if (elected) {
                mbar_expect_tx(bar, kTileBytes);
                tma_load_4d(dst, maps + mi, 0, token, h, n, bar);
                tma_load_4d(dst + kHalfBytes, maps + mi, 64, token, h, n, bar);
            }
        };
        // swizzled address of the 16-byte piece q (8 channels) of row r
        auto piece = [&](uint32_t dst, int r, int q) { return dst + (uint32_t)(q >> 3) * kHalfBytes + (uint32_t)r * 128u + (uint32_t)(((q & 7) ^ (r & 7)) << 4); };
        // 16 lanes per row (256 contiguous bytes in global memory), two rows per warp instruction; rows at
        // or beyond `nrows` are zero-filled
        auto copy_rows = [&](uint32_t dst, const __nv_bfloat16* base, int64_t st, int nrows) {
            const int q = lane & 15;
            for (int r = 2 * lw + (lane >> 4); r < 128; r += 2 * kAttnLoaderWarps) {
                const bool valid = r < nrows;
                cp_async16(piece(dst, r, q), valid ? base + (int64_t)r * st + q * 8 : safe, valid ? 16u : 0u);
            }
        };
        auto announce_copied = [&](uint32_t bar) {
            cp_async_wait_all();
            fence_proxy_async();
            asm volatile("bar.sync 2, 96;" ::: "memory");
            if (elected) mbar_arrive(bar);
        };
        // keys (which = 0) or values (1) of key tile jt into buffer buf
        auto load_kv = [&](int jt, int buf, int which) {
            const CatView& x = which ? p.xv : p.xk;
            const uint32_t dst = (which ? vs : ks) + buf * kTileBytes;
            const uint32_t bar = which ? v_full(buf) : k_full(buf);
            const int jb = tile_of(jt) * 128;
            if (jb < p.c) wait_for_earlier_kernels();          // cache rows: the previous step's result
            if (jb + 128 <= p.c) {
                const int mi = kMapKCache + which;
                if ((mask >> mi) & 1) {
                    engine_tile(dst, bar, mi, jb);
                } else {
                    copy_rows(dst, unit_base<__nv_bfloat16>(x.cache, n, h) + (int64_t)jb * x.cache.st, x.cache.st, 128);
                    announce_copied(bar);
                }
            } else if (jb >= p.c) {
                const int mi = kMapKChunk + which;
                if ((mask >> mi) & 1) {
                    engine_tile(dst, bar, mi, jb - p.c);
                } else {
                    copy_rows(dst, unit_base<__nv_bfloat16>(x.chunk, n, h) + (int64_t)(jb - p.c) * x.chunk.st, x.chunk.st, S - jb);
                    announce_copied(bar);
                }
            } else {
                // the tile straddles the end of the cache: row by row
                const int q = lane & 15;
                for (int r = 2 * lw + (lane >> 4); r < 128; r += 2 * kAttnLoaderWarps) {
                    const int j = jb + r;
                    const bool valid = j < S;
                    const __nv_bfloat16* src = !valid ? safe
                        : j < p.c ? unit_base<__nv_bfloat16>(x.cache, n, h) + (int64_t)j * x.cache.st + q * 8
                                  : unit_base<__nv_bfloat16>(x.chunk, n, h) + (int64_t)(j - p.c) * x.chunk.st + q * 8;
                    cp_async16(piece(dst, r, q), src, valid ? 16u : 0u);
                }
                announce_copied(bar);
            }
        };
        if (mask & 1u) {
            engine_tile(qs, q_full, kMapQ, r0);
        } else {
            copy_rows(qs, safe + (int64_t)r0 * p.q.st, p.q.st, p.b - r0);
            announce_copied(q_full);
        }
        // Tiles 0 and 1 go straight into the two buffers. Tile t (>= 2) goes into the buffers of tile t-2: its keys as
        // soon as S(t-2) has read the key buffer, its values as soon as PV(t-2) has read the value buffer. A tile is
        // announced (or left to the engine to announce) before this warp waits for the next buffer. (One call site
        // for all tiles: the loader's code is inlined where it is called, and there is a lot of it.)
#pragma unroll 1
        for (int t = 0; t < ntiles; ++t) {
            const int b = t & 1, ph = ((t - 2) >> 1) & 1;
#pragma unroll 1
            for (int which = 0; which < 2; ++which) {
                if (t >= 2) mbar_wait(which ? pv_done(b) : s_full(b), ph, P.status, failed, 4 + which);
                load_kv(t, b, which);
            }
        }
        if (cache_tiles == 0) wait_for_earlier_kernels();   // keeps the chain of waits unbroken
    } else if (tid == kMma) {
        // ---------------- MMA issuer: S(0), then per tile S(t) followed by PV(t-1)
        const uint32_t idesc_s = instr_desc_bf16(128, false, false);
        const uint32_t idesc_o = instr_desc_bf16(128, false, true);
        const uint64_t q0 = smem_desc_sw128(qs, 16, 1024);
        // the kk-th 16-channel step of a K-major tile: which half, then 32 bytes per step inside the row
        auto kstep = [](int kk) { return (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32u) >> 4); };
        auto issue_pv = [&](int t) {
            const int b = t & 1;
            mbar_wait(v_full(b), (t >> 1) & 1, P.status, failed, 6);
            mbar_wait(p_full(b), (t >> 1) & 1, P.status, failed, 6);
            tc_fence_after();
            // V is the MN-major operand: 64-channel blocks kHalfBytes apart, 16 keys (two 8-row groups) per step
            const uint64_t a0 = smem_desc(ps + b * kPBytes, 2048, 128), b0 = smem_desc_sw128(vs + b * kTileBytes, kHalfBytes, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) umma_ss(tmem + 256, a0 + kk * 256u, b0 + kk * 128u, idesc_o, (t | kk) != 0);
            umma_commit(pv_done(b));
        };
        mbar_wait(q_full, 0, P.status, failed, 7);
#pragma unroll 1
        for (int jt = 0; jt < ntiles; ++jt) {
            const int b = jt & 1;
            mbar_wait(k_full(b), (jt >> 1) & 1, P.status, failed, 7);
            if (jt >= 2) mbar_wait(s_free(b), ((jt >> 1) - 1) & 1, P.status, failed, 8);
            tc_fence_after();
            const uint64_t k0 = smem_desc_sw128(ks + b * kTileBytes, 16, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) umma_ss(tmem + b * 128, q0 + kstep(kk), k0 + kstep(kk), idesc_s, kk != 0);
            umma_commit(s_full(b));
            if (jt >= 1) issue_pv(jt - 1);
        }
        issue_pv(ntiles - 1);
    }
    const int rl = (warp & 3) * 32 + lane;          // row of the tile this thread works on (softmax warps)
    const int half = (warp >> 2) & 1;               // which 64 columns of the row
    const int row = r0 + rl;
    const bool live = warp < 8 && row < p.b;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    if (warp < 8) {
        // ---------------- softmax
        float m_used = 0.f, lrun = 0.f;
        const int vis = live ? p.c + row + 1 : (1 << 30);   // visible columns of this row (rows past the chunk are all zeros)
        const float sc2 = p.scale * 1.4426950408889634f;
        // the two threads of a row exchange their maxima rounded to bf16, one slot per tile parity:
        // both then derive the same reference maximum, which only has to be near the true one
        __nv_bfloat16* xmax = reinterpret_cast<__nv_bfloat16*>(xchg);   // [2 parities][2 halves][128 rows]
#pragma unroll 1
        for (int jt = 0; jt < ntiles; ++jt) {
            const int b = jt & 1;
            mbar_wait(s_full(b), (jt >> 1) & 1, P.status, failed, 9);
            tc_fence_after();
            const uint32_t s_addr = lane_base + b * 128 + half * 64;
            const int at = tile_of(jt);                   // the key tile this round works on
            const int j0 = at * 128 + half * 64;
            const bool need_mask = at * 128 + 128 > p.c + r0;
            if (jt >= 2) mbar_wait(pv_done(b), ((jt >> 1) - 1) & 1, P.status, failed, 11);   // P buffer b is free
            uint8_t* pdst = p_ptr + b * kPBytes + rl * 16;
            // One sweep over this thread's 64 logits: P = exp2(s - m) in bf16 into the A-operand layout
            // [key group][row][8 keys], with the reference maximum m carried over from the earlier tiles,
            // and the tile's own maximum on the side. Only if that maximum turns out to exceed m by more
            // than the threshold (always for the first tile, rarely later) is m raised, O rescaled and
            // the sweep repeated; a P that overflowed in the discarded sweep is simply overwritten.
            float lsum = 0.f;
            // (compiled twice: tiles that the causal limit crosses test every column, the others none)
            auto sweep = [&](auto masked, float& tmax) {
                constexpr bool kMasked = decltype(masked)::value;
                float sum = 0.f;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(s_addr + c0, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int x = 0; x < 8; x += 2) {
                            const int ja = j0 + c0 + e + x;
                            // one FMA per logit: exp2(s * scale - m); the maximum is tracked on the raw logits
                            // and scaled once per tile (the scale is positive)
                            const float ra = __uint_as_float(v[e + x]), rb = __uint_as_float(v[e + x + 1]);
                            float pa = exp2f(fmaf(ra, sc2, -m_used)), pb = exp2f(fmaf(rb, sc2, -m_used));
                            if (kMasked && ja >= vis) pa = 0.f; else tmax = fmaxf(tmax, ra);
                            if (kMasked && ja + 1 >= vis) pb = 0.f; else tmax = fmaxf(tmax, rb);
                            const __nv_bfloat162 pr = __floats2bfloat162_rn(pa, pb);
                            pk[x >> 1] = *reinterpret_cast<const uint32_t*>(&pr);
                            // the row sum takes the terms as rounded for the PV product: with a few dominant keys the
                            // rounding of P then cancels in O / sum instead of showing up as a 0.4 % error
                            sum += __low2float(pr) + __high2float(pr);
                        }
                        *reinterpret_cast<uint4*>(pdst + ((half * 64 + c0 + e) >> 3) * 2048) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                return sum;
            };
            // the first tile has no reference maximum yet, so its first pass only looks for one
            auto max_only = [&](float& tmax) {
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(s_addr + c0, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (!need_mask || j0 + c0 + e < vis) tmax = fmaxf(tmax, __uint_as_float(v[e]));
                }
            };
#pragma unroll 1
            for (int attempt = 0; attempt < 2; ++attempt) {
                float tmax = -INFINITY;
                if (jt == 0 && attempt == 0) max_only(tmax);
                else lsum = need_mask ? sweep(std::true_type{}, tmax) : sweep(std::false_type{}, tmax);
                if (attempt == 1) break;
                const __nv_bfloat16 mine = __float2bfloat16_rn(tmax * sc2);
                xmax[b * 256 + half * 128 + rl] = mine;
                asm volatile("bar.sync 1, 256;" ::: "memory");
                const float mt = fmaxf(__bfloat162float(mine), __bfloat162float(xmax[b * 256 + (half ^ 1) * 128 + rl]));
                // the first tile worked on holds a key every row sees (the chunk's first, or key 0), so mt is finite there
                const bool bump = jt == 0 || mt > m_used + kRescaleThreshold;
                if (!__any_sync(0xffffffffu, bump)) break;
                if (jt > 0) {
                    const float f = bump ? exp2f(m_used - mt) : 1.f;
                    mbar_wait(pv_done((jt - 1) & 1), ((jt - 1) >> 1) & 1, P.status, failed, 10);
                    tc_fence_after();
#pragma unroll
                    for (int c0 = 0; c0 < 64; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(lane_base + 256 + half * 64 + c0, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * f);
                        tmem_st32(lane_base + 256 + half * 64 + c0, v);
                    }
                    tmem_st_wait();
                    lrun *= f;
                }
                if (bump) m_used = mt;
            }
            lrun += lsum;
            tc_fence_before();
            mbar_arrive(s_free(b));      // this thread's reads of S[b] are complete (wait::ld above)
            fence_proxy_async();
            mbar_arrive(p_full(b));
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");      // every exchange slot has been read: the sums reuse the space
        // the last PV has updated O
        mbar_wait(pv_done((ntiles - 1) & 1), ((ntiles - 1) >> 1) & 1, P.status, failed, 12);
        tc_fence_after();
        xchg[half * 128 + rl] = lrun;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        const float ltot = lrun + xchg[(half ^ 1) * 128 + rl];
        const float inv = 1.f / ltot;
        __nv_bfloat16* orow = unit_base_mut<__nv_bfloat16>(p.o, n, h) + (int64_t)(live ? row : 0) * p.o.st + half * 64;
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(lane_base + 256 + half * 64 + c0, v);
            tmem_ld_wait();
            if (live) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv);
                    o.y = pack_bf16(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv);
                    o.z = pack_bf16(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv);
                    o.w = pack_bf16(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv);
                    *reinterpret_cast<uint4*>(orow + c0 + e) = o;
                }
            }
        }
        if (live && p.lse && half == 0) p.lse[(int64_t)u * p.lse_stride + row] = (m_used + log2f(ltot)) * 0.6931471805599453f;
    }
    if (maps_fresh) {
        // (the persistent kernel: its CTA goes on to other work in this shared memory)
        tc_fence_before();
        __syncthreads();
        if (warp == kMma / 32 && (tid & 31) < 13) mbar_inval(bar0 + 8 * (tid & 31));
    }
}

__global__ void __launch_bounds__(kAttnThreads, 1) attention_tc_kernel(const __grid_constant__ TcAttnParams P) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t tmem_slot;
    const uint32_t tmem = cta_tmem_acquire(&tmem_slot);
    attention_body(P, P.maps, false, smem, tmem, blockIdx.x, blockIdx.y);
    cta_tmem_release(tmem);
}

// Eq. 1 for a chunk of ONE query (the generation stage) on the CUDA cores: a 128-row MMA tile would hold one live row.
// The step is a chain of memory latencies and every CTA runs this code exactly once, so it is written for few
// round trips and few instructions (short rolled loops: straight-line code that runs once costs its own fetch):
// the work of a unit is spread over four warps, a quarter of the keys each; a warp brings its key and value rows
// into shared memory with one burst of 16-byte async copies, then scores and accumulates from there. A lane owns
// four channels; the four warps' (maximum, sum, output) triples meet in shared memory.
constexpr int kDecodeWarpsPerUnit = 4;
constexpr int kDecodeUnitsPerCta = kThreads / 32 / kDecodeWarpsPerUnit;
constexpr int kDecodeRows = 33;                                        // keys per warp
constexpr int kDecodeMaxKeys = kDecodeRows * kDecodeWarpsPerUnit;      // 132: a cache of 128 slots and the query's own key

__device__ __forceinline__ void decode_attention_body(const TcAttnParams& P, uint8_t* smem, int first_unit) {
    const AttnParams& p = P.base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int u = first_unit + warp / kDecodeWarpsPerUnit, part = warp % kDecodeWarpsPerUnit;
    const bool live = u < p.units;
    const int n = live ? u / p.heads : 0, h = live ? u % p.heads : 0;
    const int S = p.c + 1;
    const int per = (S + kDecodeWarpsPerUnit - 1) / kDecodeWarpsPerUnit;
    const int j_begin = part * per, j_end = live ? min(S, j_begin + per) : j_begin;   // this warp's keys
    const int nk = j_end - j_begin;
    uint8_t* rows = smem + warp * (2 * kDecodeRows * 256);            // [keys: nk rows][values: nk rows at kDecodeRows], 256 bytes each
    const uint32_t rows_a = smem_u32(rows);
    float* xch = reinterpret_cast<float*>(smem + (kThreads / 32) * (2 * kDecodeRows * 256));
    auto f4 = [](uint2 x, float (&o)[4]) {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.y));
        o[0] = a.x; o[1] = a.y; o[2] = b.x; o[3] = b.y;
    };
    float q[4];
    f4(live ? *reinterpret_cast<const uint2*>(unit_base<__nv_bfloat16>(p.q, n, h) + 4 * lane) : make_uint2(0u, 0u), q);
    wait_for_earlier_kernels();          // the cache rows are the previous step's result
    {
        // 16 lanes per row, two rows per instruction; rows of the cache, then (the last key) the chunk's row
        const __nv_bfloat16* kc = unit_base<__nv_bfloat16>(p.xk.cache, n, h) + 8 * (lane & 15);
        const __nv_bfloat16* vc = unit_base<__nv_bfloat16>(p.xv.cache, n, h) + 8 * (lane & 15);
        const __nv_bfloat16* kn = unit_base<__nv_bfloat16>(p.xk.chunk, n, h) + 8 * (lane & 15);
        const __nv_bfloat16* vn = unit_base<__nv_bfloat16>(p.xv.chunk, n, h) + 8 * (lane & 15);
#pragma unroll 1
        for (int r = lane >> 4; r < nk; r += 2) {
            const int j = j_begin + r;
            const uint32_t dst = rows_a + r * 256 + (lane & 15) * 16;
            cp_async16(dst, j < p.c ? kc + (int64_t)j * p.xk.cache.st : kn, 16u);
            cp_async16(dst + kDecodeRows * 256, j < p.c ? vc + (int64_t)j * p.xv.cache.st : vn, 16u);
        }
        cp_async_wait_all();
        __syncwarp();
    }
    const float sc2 = p.scale * 1.4426950408889634f;
    // scores: lane l keeps the score of keys l and 32 + l of this warp
    float s0 = -INFINITY, s1 = -INFINITY;
#pragma unroll 1
    for (int r = 0; r < nk; ++r) {
        float kf[4];
        f4(*reinterpret_cast<const uint2*>(rows + r * 256 + lane * 8), kf);
        float d = fmaf(q[0], kf[0], fmaf(q[1], kf[1], fmaf(q[2], kf[2], q[3] * kf[3])));
#pragma unroll
        for (int o = 16; o; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        d *= sc2;
        if ((r & 31) == lane) { if (r < 32) s0 = d; else s1 = d; }
    }
    float m_w = fmaxf(s0, s1);
#pragma unroll
    for (int o = 16; o; o >>= 1) m_w = fmaxf(m_w, __shfl_xor_sync(0xffffffffu, m_w, o));
    const float p0 = lane < nk ? exp2f(s0 - m_w) : 0.f, p1 = 32 + lane < nk ? exp2f(s1 - m_w) : 0.f;
    float l_w = p0 + p1;
#pragma unroll
    for (int o = 16; o; o >>= 1) l_w += __shfl_xor_sync(0xffffffffu, l_w, o);
    float o4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
    for (int r = 0; r < nk; ++r) {
        const float pj = __shfl_sync(0xffffffffu, r < 32 ? p0 : p1, r & 31);
        float vf[4];
        f4(*reinterpret_cast<const uint2*>(rows + (kDecodeRows + r) * 256 + lane * 8), vf);
#pragma unroll
        for (int e = 0; e < 4; ++e) o4[e] = fmaf(pj, vf[e], o4[e]);
    }
    // the four warps of a unit meet: [warp][maximum, sum, -, -, 128 outputs]
    constexpr int kRec = 4 + kD;
    float* mine = xch + warp * kRec;
    if (lane == 0) { mine[0] = nk > 0 ? m_w : -INFINITY; mine[1] = l_w; }
    *reinterpret_cast<float4*>(mine + 4 + 4 * lane) = make_float4(o4[0], o4[1], o4[2], o4[3]);
    __syncthreads();
    if (live && part == 0) {
        const float* base = xch + (warp / kDecodeWarpsPerUnit) * kDecodeWarpsPerUnit * kRec;
        float m_all = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarpsPerUnit; ++w) m_all = fmaxf(m_all, base[w * kRec]);
        float l_all = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int w = 0; w < kDecodeWarpsPerUnit; ++w) {
            const float* src = base + w * kRec;
            const float mw = src[0];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - m_all);
            l_all += src[1] * f;
            const float4 ow = *reinterpret_cast<const float4*>(src + 4 + 4 * lane);
            o[0] = fmaf(ow.x, f, o[0]); o[1] = fmaf(ow.y, f, o[1]); o[2] = fmaf(ow.z, f, o[2]); o[3] = fmaf(ow.w, f, o[3]);
        }
        const float inv = 1.f / l_all;
        uint2 out;
        out.x = pack_bf16(o[0] * inv, o[1] * inv);
        out.y = pack_bf16(o[2] * inv, o[3] * inv);
        reinterpret_cast<uint2*>(unit_base_mut<__nv_bfloat16>(p.o, n, h))[lane] = out;
        if (p.lse && lane == 0) p.lse[(int64_t)u * p.lse_stride] = (m_all + log2f(l_all)) * 0.6931471805599453f;
    }
}

// ------------------------------------------------------------------ one chunk step, one launch
// Step 3 (attention with the OLD cache) and Steps 4-5 (the new cache) of Algorithm 2 read the same
// inputs and do not depend on each other, so their CTAs share one grid: every CTA fills an SM by
// itself, the attention CTAs differ in length (2..5 key tiles), and a mixed grid lets the block
// scheduler pack all of them onto the 148 SMs instead of two launches of 128 CTAs each.
// Block order: the attention tiles estimated to outlast a compress CTA first (only where the grid is more than
// two waves of CTAs), then the compress CTAs, then the remaining attention tiles, longest first.
struct TcStepParams {
    TcAttnParams attn;
    TcCompressParams comp;
    TcTileMaps tiles;
    int qtiles, n_attn_first, n_attn, comp_per_unit;   // comp_per_unit = parts * slot_blocks
    int decode;                                        // 1: chunks of one query, attention by decode_attention_body (a warp per unit)
    // position in the item list of a persistent launch (sequence_tc_kernel)
    int items_per_unit, item_end, finished_target;     // finished_target: items of a unit up to and including this step
};

// Work item `idx` of one chunk step, in the order above. (Each body appears once: the kernel's code is several times the
// size of an SM's instruction cache as it is, and code that has to be fetched is time the CTA spends waiting.)
__device__ __forceinline__ void step_item(const TcStepParams& P, uint8_t* smem, uint32_t tmem, bool cache_cg, int idx) {
    const int units = P.attn.base.units;
    const int n_comp = P.comp.pair ? P.comp.pairs : units * P.comp_per_unit;
    const bool is_comp = idx >= P.n_attn_first && idx < P.n_attn_first + n_comp;
    if (is_comp) {
        idx -= P.n_attn_first;
        if (P.comp.pair) {
            compress_pair_body(P.comp, &P.attn.maps[kMapVCache], &P.tiles, smem, tmem, idx);
        } else {
            const int u = idx / P.comp_per_unit, rem = idx % P.comp_per_unit;
            compress_body<true>(P.comp, &P.tiles, smem, tmem, cache_cg, rem % P.comp.parts, rem / P.comp.parts, u);
        }
    } else {
        if (idx >= P.n_attn_first) idx -= n_comp;       // the attention items after the compress CTAs continue the first ones' numbering
        if (P.decode) decode_attention_body(P.attn, smem, idx * kDecodeUnitsPerCta);
        else attention_body(P.attn, P.attn.maps, false, smem, tmem, P.qtiles - 1 - idx / units, idx % units);
    }
}

__global__ void __launch_bounds__(kAttnThreads, 1) chunk_step_tc_kernel(const __grid_constant__ TcStepParams P) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t tmem_slot;
    overlap_with_neighbours();
    const uint32_t tmem = cta_tmem_acquire(&tmem_slot);
    step_item(P, smem, tmem, false, blockIdx.x);     // the bodies wait for the earlier kernels where they need them
    cta_tmem_release(tmem);
}

// ------------------------------------------------------------------ the whole chunk loop, one launch
// A persistent grid (one CTA per SM) works through the steps of Algorithm 2 as ONE list of work items,
// step after step and unit after unit inside a step, pulled from a counter. Steps of different units
// are independent, so there is no device-wide barrier: an item of step n waits only until ITS unit's
// cache holds the result of step n-1 (a per-unit step counter), and the CTA that completes the last
// item of a (step, unit) pair rebuilds that unit's cache from the partial blends and publishes the
// counter. While the slowest unit of a step is still busy, the other SMs already run the next step of
// the units that are done; launch gaps, TMEM set-up and the per-step tail of the block scheduler go.
// Items are handed out in list order and only ever wait for items earlier in the list, which a
// running CTA has already taken: every wait ends whether or not all CTAs are resident at once.
struct TcSeqParams {
    const TcStepParams* steps;   // device
    int n_steps, total_items;
    int* work;                   // next item of the list; zeroed before the launch
    int* finished;               // [units] items completed so far; zeroed before the launch
    int* version;                // [units] steps whose cache update is complete; zeroed before the launch
    int* status;
};

// New cache of unit u from the partial blends and row sums (Eq. 7 after Eq. 4-5), by one CTA of 384
// threads. The partial sets (64 KB each, channel-major) come in through the copy engine, up to three at
// a time; with more than three the earlier ones are folded into the first buffer. Sums run over the
// sets in order, as in finalize_tile. A thread then owns one slot and eight channels: it reads along
// channels (stride = one row of slots, its lane's bank), scales by 1/(s + eps) and stores 16 bytes.
__device__ __forceinline__ void finalize_unit(const TcCompressParams& P, uint8_t* smem, int u) {
    const CompressParams& p = P.base;
    const int n = u / p.heads, h = u % p.heads;
    constexpr int kSet = kSlots * kD;                             // floats per partial set
    float* bufs = reinterpret_cast<float*>(smem);                 // [3][128 channels][128 slots]
    float* inv_s = bufs + 3 * kSet;
    uint64_t* bar = reinterpret_cast<uint64_t*>(inv_s + kSlots);
    volatile int* failed = reinterpret_cast<volatile int*>(bar + 1);
    const uint32_t bar_a = smem_u32(bar), bufs_a = smem_u32(bufs);
    const int tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(bar_a, 1);
        *failed = 0;
        fence_barrier_init();
    }
    __syncthreads();
    uint32_t phase = 0;
    for (int sb = 0; sb < P.slot_blocks; ++sb) {
        const int64_t base = ((int64_t)u * P.slot_blocks + sb) * P.part_stride;
        if (tid < kSlots) {
            float sum = 0.f;
            for (int pt = 0; pt < P.parts; ++pt) sum += __ldcg(P.part_s + (base + pt) * kSlots + tid);
            sum = sb * kSlots + tid < p.prot ? 1.f : sum + p.eps;
            inv_s[tid] = 1.f / sum;
            p.s[(int64_t)u * p.M + sb * kSlots + tid] = sum;
        }
        __syncthreads();
        for (int mat = 0; mat < 2; ++mat) {
            int live = 0;                                         // buffers to add up at the end
            for (int pt = 0; pt < P.parts;) {
                const int first_buf = pt == 0 ? 0 : 1;
                const int cnt = min(P.parts - pt, 3 - first_buf);
                if (tid == 0) {
                    // the buffers' earlier accesses and the partials' arrival, before the copy engine's
                    asm volatile("fence.proxy.async;" ::: "memory");
                    mbar_expect_tx(bar_a, (uint32_t)cnt * kSet * 4u);
                    for (int i = 0; i < cnt; ++i) {
                        const float* src = P.part_U + ((base + pt + i) * 2 + mat) * kSet;
                        for (uint32_t piece = 0; piece < kSet * 4u; piece += kStageBytes)
                            bulk_load(bufs_a + (first_buf + i) * kSet * 4u + piece, reinterpret_cast<const uint8_t*>(src) + piece,
                                      kStageBytes, bar_a);
                    }
                }
                mbar_wait(bar_a, phase, P.status, failed, 21);
                phase ^= 1;
                pt += cnt;
                live = first_buf + cnt;
                if (pt < P.parts) {                               // more sets than buffers: fold into the first
                    for (int i4 = tid; i4 < kSet / 4; i4 += kAttnThreads) {
                        float4 acc = reinterpret_cast<float4*>(bufs)[i4];
                        for (int b = 1; b < live; ++b) {
                            const float4 v = reinterpret_cast<const float4*>(bufs + b * kSet)[i4];
                            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                        }
                        reinterpret_cast<float4*>(bufs)[i4] = acc;
                    }
                    __syncthreads();
                }
            }
            const View& out = mat ? p.v_out : p.k_out;
            for (int idx = tid; idx < (kD / 8) * kSlots; idx += kAttnThreads) {
                const int g = idx / kSlots, sl = idx % kSlots;
                const float* src = bufs + (g * 8) * kSlots + sl;
                float v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = 0.f;
                for (int b = 0; b < live; ++b) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] += src[b * kSet + e * kSlots];
                }
                const float inv = inv_s[sl];
                uint4 o;
                o.x = pack_bf16(v[0] * inv, v[1] * inv);
                o.y = pack_bf16(v[2] * inv, v[3] * inv);
                o.z = pack_bf16(v[4] * inv, v[5] * inv);
                o.w = pack_bf16(v[6] * inv, v[7] * inv);
                *reinterpret_cast<uint4*>(unit_base_mut<__nv_bfloat16>(out, n, h) + (int64_t)(sb * kSlots + sl) * out.st + g * 8) = o;
            }
            __syncthreads();
        }
    }
    if (tid == 0) mbar_inval(bar_a);
}

__global__ void __launch_bounds__(kAttnThreads, 1) sequence_tc_kernel(const __grid_constant__ TcSeqParams Q) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t tmem_slot;
    __shared__ int item_s, last_s;
    const uint32_t tmem = cta_tmem_acquire(&tmem_slot);
    int n = 0;
    // a thread-private copy: parameters read through a global pointer cannot be kept in registers
    // across the bodies' stores, and the bodies read them inside their hot loops
    TcStepParams P = Q.steps[0];
    while (true) {
        if (threadIdx.x == 0) {
            // after a wait has run out anywhere the results are void: stop handing out work
            item_s = *reinterpret_cast<volatile int*>(Q.status) == 0 ? atomicAdd(Q.work, 1) : Q.total_items;
        }
        __syncthreads();
        const int item = item_s;
        __syncthreads();
        if (item >= Q.total_items) break;
        while (n + 1 < Q.n_steps && item >= P.item_end) P = Q.steps[++n];
        const int local = item - (P.item_end - P.items_per_unit * P.attn.base.units);
        const int u = local / P.items_per_unit;
        int r = local % P.items_per_unit;
        if (n > 0) {
            // unit u's cache must hold the result of step n-1 (bounded wait; acquire, then the CTA barrier,
            // orders every thread's reads of the cache and of nothing older after the publication)
            if (threadIdx.x == 0) {
                bool ok = false;
                for (uint32_t i = 0; i < (1u << 22); ++i) {
                    int seen;
                    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(Q.version + u) : "memory");
                    if (seen >= n) { ok = true; break; }
                    __nanosleep(32);
                }
                if (!ok) atomicCAS(Q.status, 0, 20);
                __threadfence();
            }
            __syncthreads();
        }
        // within a unit: compress CTAs first (the longest), then the attention tiles, longest first
        // (cache rows rewritten by other SMs earlier in this same kernel are read around L1)
        if (r < P.comp_per_unit) compress_body<false>(P.comp, nullptr, smem, tmem, n > 0, r % P.comp.parts, r / P.comp.parts, u);
        else attention_body(P.attn, Q.steps[n].attn.maps, true, smem, tmem, P.qtiles - 1 - (r - P.comp_per_unit), u);
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();                                        // this item's stores, then the count
            const int done = atomicAdd(Q.finished + u, 1) + 1;
            last_s = done == P.finished_target;
            if (last_s) __threadfence();
        }
        __syncthreads();
        if (last_s) {
            finalize_unit(P.comp, smem, u);
            if (threadIdx.x == 0) {
                __threadfence();
                asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(Q.version + u), "r"(n + 1) : "memory");
            }
        }
    }
    cta_tmem_release(tmem);
}

constexpr int kMaxSeqSteps = 256;   // steps one persistent launch can hold

struct Plan {
    int n_tile, tiles, parts, tiles_per_part, stages, rows_pad;
    size_t smem;
    double cta_us;   // estimated duration of one compress CTA
};

int parts_cap(int units, int slot_blocks) {
    const int pairs = units * slot_blocks;
    return (600 + pairs - 1) / pairs;
}

int tile_rows_alloc(int n_tile, int k) { return (n_tile + k - 1 + 7) / 8 * 8; }    // halves of a tile stay on 1024-byte boundaries

size_t smem_bytes(int n_tile, int k, int stages) {
    return 1024 + (size_t)stages * kStageBytes + 2 * 256 * (size_t)tile_rows_alloc(n_tile, k) + (2 * stages + 4) * 8 + 16;
}

// Tile width and CTA count: fewest waves of 148 SMs, then least padded work.
// Cost model from measured CTA timelines (microseconds): a fixed part (set-up, key staging, partial
// stores), and per position tile one ring stage per (tap, channel half) that takes the longer of the
// weight copy (0.37) and its eight MMAs (N/2 cycles each), plus epilogue and blends. A stand-alone
// launch is charged by waves of 148 SMs; CTAs that share a grid with attention CTAs (`fused`) are
// charged by their total SM time, which favours wider tiles (fewer CTAs, overheads paid less often).
bool make_plan(int S, int k, int halves, int units, int slot_blocks, bool fused, Plan* out) {
    double best = 1e30;
    const int cap = parts_cap(units, slot_blocks);
    for (int n_tile = 224; n_tile >= 64; n_tile -= 32) {
        int stages = 4;
        while (stages >= 2 && smem_bytes(n_tile, k, stages) > (size_t)kMaxSmem) --stages;
        if (stages < 2 || (size_t)stages * kStageBytes < (size_t)n_tile * kSlots * 2) continue;
        const int tiles = (S + n_tile - 1) / n_tile;
        for (int parts = 1; parts <= tiles && parts <= cap; ++parts) {
            const int tpp = (tiles + parts - 1) / parts;
            const int parts_eff = (tiles + tpp - 1) / tpp;
            const long ctas = (long)units * slot_blocks * parts_eff;
            const long waves = (ctas + 147) / 148;
            const double stage_us = std::max(0.37, n_tile * 0.5 * 8.0 / 1965.0);
            const double cta_us = 4.0 + tpp * (k * halves * stage_us + 3.5);
            const double cost = (fused ? ctas * cta_us / 148.0 + 0.5 * cta_us : waves * cta_us) + (stages < 4 ? 0.05 : 0.0);
            if (cost < best) {
                best = cost;
                *out = Plan{n_tile, tiles, parts_eff, tpp, stages, tile_rows_alloc(n_tile, k), smem_bytes(n_tile, k, stages), cta_us};
            }
        }
    }
    return best < 1e30;
}

}  // namespace

int simt_write_weights(const float* R, const float* s, float* W, int64_t rows, int S, cudaStream_t st);

bool tensor_config_supported(const lococo_config* c) {
    if (c->dtype != LOCOCO_BF16 || c->head_dim != kD) return false;
    if (c->M % kSlots != 0) return false;
    Plan pl;
    return make_plan(c->M + c->max_chunk, c->k, c->c_in / 128, c->batch * c->heads, c->M / kSlots, false, &pl);
}

void tensor_layout_workspace(lococo_handle* h, size_t* off) {
    if (!h->use_tensor) return;
    const lococo_config& c = h->cfg;
    auto align = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t sets = c.weights_per_head ? c.heads : 1;
    const int SB = c.M / kSlots;
    const int Smax = c.M + c.max_chunk;
    const int max_parts = std::min(parts_cap(h->units, SB), (Smax + 63) / 64);
    h->off_gimage = *off;
    *off = align(*off + sets * (size_t)c.M * c.c_in * c.k * 2);
    h->off_part = *off;
    *off = align(*off + (size_t)h->units * SB * max_parts * (2 * kSlots * kD + kSlots) * sizeof(float));
    h->off_steps = *off;
    *off = align(*off + (size_t)kMaxSeqSteps * sizeof(TcStepParams));
    h->off_sync = *off;
    *off = align(*off + (size_t)(64 + 2 * h->units) * sizeof(int));   // item counter, then per unit: finished, version
    h->off_alt_k = *off;
    *off = align(*off + (size_t)h->units * c.M * kD * 2);
    h->off_alt_v = *off;
    *off = align(*off + (size_t)h->units * c.M * kD * 2);
    h->off_merge = *off;
    *off = align(*off + (size_t)h->units * SB * 2 * sizeof(int));   // per (unit, slot block): CTAs arrived, partial sets stored
}

int tensor_pack_weights(lococo_handle* h, const void* G, cudaStream_t st) {
    const lococo_config& c = h->cfg;
    const int sets = c.weights_per_head ? c.heads : 1;
    const int64_t total = (int64_t)sets * c.M * c.c_in * c.k;
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, 8192);
    pack_image_kernel<<<blocks, 256, 0, st>>>((const __nv_bfloat16*)G, (__nv_bfloat16*)(h->ws + h->off_gimage), sets, c.M,
                                              c.c_in, c.k);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

bool tensor_compress_supported(const lococo_handle* h, const CompressParams& p) {
    Plan pl;
    return h->use_tensor && p.S >= 1 && make_plan(p.S, p.k, p.c_in / 128, p.units, p.M / kSlots, false, &pl);
}


// ---- tensor maps
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled() {
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

// View [batch, heads, tokens, 128] of bf16, `tokens` rows valid (rows beyond, or before row 0, read as zeros): boxes of
// `box_rows` tokens x 64 channels in the 128-byte swizzle.
static bool make_rows_map(CUtensorMap* map, const View& v, int tokens, int heads, int batch, int box_rows) {
    EncodeTiledFn fn = encode_tiled();
    if (!fn || tokens < 1 || box_rows < 1 || box_rows > 256) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)batch};
    cuuint64_t strides[3] = {(cuuint64_t)v.st * 2, (cuuint64_t)v.sh * 2, (cuuint64_t)v.sb * 2};
    // a dimension of extent 1 never uses its stride: give it a harmless one
    if (heads == 1) strides[1] = strides[0] * (cuuint64_t)tokens;
    if (batch == 1) strides[2] = strides[1] * (cuuint64_t)heads;
    for (cuuint64_t st : strides)
        if (st == 0 || st % 16 != 0 || st >= ((cuuint64_t)1 << 40)) return false;
    if (v.st < 0 || v.sh < 0 || v.sb < 0 || reinterpret_cast<uintptr_t>(v.ptr) % 16 != 0) return false;
    const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, v.ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
static bool make_tile_map(CUtensorMap* map, const View& v, int tokens, int heads, int batch) {
    return make_rows_map(map, v, tokens, heads, batch, 128);
}

// The tile maps of a compress launch whose tiling is already in P: whole-tile boxes of the cache and of the chunk, and
// for each tile that holds the seam a pair of boxes with the heights of its two parts. Any refusal: async copies.
static void fill_tile_maps(TcCompressParams* P, TcTileMaps* T) {
    const CompressParams& p = P->base;
    const int batch = p.units / p.heads, pad = (p.k - 1) / 2, rows = P->n_tile + p.k - 1, c = p.xk.c, b = p.S - c;
    P->tile_maps = 0;
    P->out_maps = 0;
    P->seam_h1[0] = P->seam_h1[1] = 0;
    if (b < 1) return;
    bool ok = make_rows_map(&T->m[kTmKChunk], p.xk.chunk, b, p.heads, batch, rows) &&
              make_rows_map(&T->m[kTmVChunk], p.xv.chunk, b, p.heads, batch, rows);
    if (ok && c > 0)
        ok = make_rows_map(&T->m[kTmKCache], p.xk.cache, c, p.heads, batch, rows) &&
             make_rows_map(&T->m[kTmVCache], p.xv.cache, c, p.heads, batch, rows);
    int seams = 0;
    for (int t = 0; ok && c > 0 && t < P->tiles; ++t) {
        const int h1 = std::max(0, std::min(rows, c - (t * P->n_tile - pad)));
        if (h1 == 0 || h1 == rows || h1 == P->seam_h1[0] || h1 == P->seam_h1[1]) continue;
        if (seams == 2) break;                       // (cannot happen with one seam; such a tile would be staged by async copies)
        CUtensorMap* m = &T->m[kTmSeam + 4 * seams];
        ok = make_rows_map(m + 0, p.xk.cache, c, p.heads, batch, h1) && make_rows_map(m + 1, p.xk.chunk, b, p.heads, batch, rows - h1) &&
             make_rows_map(m + 2, p.xv.cache, c, p.heads, batch, h1) && make_rows_map(m + 3, p.xv.chunk, b, p.heads, batch, rows - h1);
        P->seam_h1[seams++] = h1;
    }
    if (ok) P->tile_maps = 1;
    else P->seam_h1[0] = P->seam_h1[1] = 0;
    // the output cache, for the CTAs that write their rows themselves
    P->out_maps = make_rows_map(&T->m[kTmKOut], p.k_out, p.M, p.heads, batch, kSlots) &&
                  make_rows_map(&T->m[kTmVOut], p.v_out, p.M, p.heads, batch, kSlots);
}

static bool build_compress_params(lococo_handle* h, const CompressParams& p, bool fused, TcCompressParams* out,
                                  double* cta_us = nullptr) {
    const int SB = p.M / kSlots;
    Plan pl;
    if (!make_plan(p.S, p.k, p.c_in / 128, p.units, SB, fused, &pl)) return false;
    const int Smax = h->cfg.M + h->cfg.max_chunk;
    const int max_parts = std::min(parts_cap(h->units, SB), (Smax + 63) / 64);
    if (pl.parts > max_parts) return false;
    TcCompressParams P{};
    P.base = p;
    P.gimage = reinterpret_cast<const __nv_bfloat16*>(h->ws + h->off_gimage);
    P.part_U = reinterpret_cast<float*>(h->ws + h->off_part);
    P.part_s = P.part_U + (size_t)p.units * SB * max_parts * 2 * kSlots * kD;
    P.R_store = p.W_out ? p.R : nullptr;
    P.status = reinterpret_cast<int*>(h->ws + h->off_status);
    P.merge_count = reinterpret_cast<int*>(h->ws + h->off_merge);
    P.n_tile = pl.n_tile; P.tiles = pl.tiles; P.parts = pl.parts; P.tiles_per_part = pl.tiles_per_part;
    P.part_stride = fused ? max_parts : pl.parts;   // fixed regions where steps with different plans share a launch
    P.halves = p.c_in / 128; P.stages = pl.stages; P.rows_pad = pl.rows_pad; P.slot_blocks = SB;
    *out = P;
    if (cta_us) *cta_us = pl.cta_us;
    return true;
}

// Launch that lets the kernel begin while its predecessor in the stream is still draining; the kernel
// itself waits (wait_for_earlier_kernels) before it touches anything the predecessor produces.
template <typename Param>
static cudaError_t launch_overlapped(void (*kernel)(Param), dim3 grid, dim3 block, size_t smem, cudaStream_t st, const Param& arg,
                                     bool overlap = true) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, arg);
}


// The dynamic shared-memory limit of a kernel is a per-device attribute: it is set on the first launch on each device.
template <typename Kernel>
static bool smem_limit_set(Kernel kernel, int bytes, bool (&done)[64]) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (!done[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
        done[dev] = true;
    }
    return true;
}

// finalize (+ optional mixing-weight output) after the compress CTAs of either launch form
static int finish_compress(const TcCompressParams& P, cudaStream_t st) {
    const CompressParams& p = P.base;
    int launches = 0;
    dim3 fgrid(p.M / 32, kD / 32, p.units);
    if (launch_overlapped(finalize_parts_kernel, fgrid, dim3(256), 0, st, P) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    ++launches;
    if (p.W_out) {
        const int r = simt_write_weights(p.R, p.s, p.W_out, (int64_t)p.units * p.M, p.S, st);
        if (r < 0) return -1;
        launches += r;
    }
    return launches;
}

int tensor_compress(lococo_handle* h, const CompressParams& p, cudaStream_t st) {
    TcCompressParams P;
    if (!build_compress_params(h, p, false, &P)) return -1;
    static bool attr_set[64] = {};
    if (!smem_limit_set(compress_tc_kernel, kMaxSmem, attr_set)) return -1;
    dim3 grid(P.parts, P.slot_blocks, p.units);
    TcCompressLaunch launch{};
    launch.c = P;
    fill_tile_maps(&launch.c, &launch.t);
    prof_begin(p.prof, 0, st);
    // the full 227 KB keeps one CTA per SM, so a CTA always finds its 512 TMEM columns free
    compress_tc_kernel<<<grid, kThreads, kMaxSmem, st>>>(launch);
    const bool ok = cudaGetLastError() == cudaSuccess;
    prof_end(p.prof, st);
    if (!ok) return -1;
    const int r = finish_compress(P, st);
    return r < 0 ? -1 : 1 + r;
}

// ---- tensor maps of the attention operands
static void fill_attention_maps(TcAttnParams* P) {
    const AttnParams& a = P->base;
    const int batch = a.units / a.heads;
    P->tma_mask = 0;
    if (make_tile_map(&P->maps[kMapQ], a.q, a.b, a.heads, batch)) P->tma_mask |= 1u << kMapQ;
    if (make_tile_map(&P->maps[kMapKChunk], a.xk.chunk, a.b, a.heads, batch)) P->tma_mask |= 1u << kMapKChunk;
    if (make_tile_map(&P->maps[kMapVChunk], a.xv.chunk, a.b, a.heads, batch)) P->tma_mask |= 1u << kMapVChunk;
    if (a.c >= 128) {
        if (make_tile_map(&P->maps[kMapKCache], a.xk.cache, a.c, a.heads, batch)) P->tma_mask |= 1u << kMapKCache;
        if (make_tile_map(&P->maps[kMapVCache], a.xv.cache, a.c, a.heads, batch)) P->tma_mask |= 1u << kMapVCache;
    }
}

static bool build_step_params(lococo_handle* h, const AttnParams& a, const CompressParams& p, TcStepParams* out) {
    TcStepParams P{};
    double comp_us = 0.0;
    if (!build_compress_params(h, p, true, &P.comp, &comp_us)) return false;
    fill_tile_maps(&P.comp, &P.tiles);
    P.attn.base = a;
    P.attn.status = P.comp.status;
    fill_attention_maps(&P.attn);
    P.qtiles = (a.b + 127) / 128;
    P.n_attn = P.qtiles * a.units;
    // longest first: the attention tiles estimated to outlast a compress CTA (7 us fixed + 2.4 us per
    // key tile, from measured timelines), then the compress CTAs, then the remaining attention tiles
    int longer = 0;
    for (int t = P.qtiles - 1; t >= 0; --t) {
        const int cols = a.c + std::min(a.b, (t + 1) * 128);
        if (7.0 + 2.4 * ((cols + 127) / 128) > comp_us) ++longer; else break;
    }
    P.comp_per_unit = P.comp.parts * P.comp.slot_blocks;
    // With at most two waves of CTAs the step is not a packing problem: its length is set by the chain through the
    // compress CTAs that hold the cache rows (wait for the previous step, conv, merge of the unit's partial blends),
    // so those start first and the attention CTAs fill in behind them (cfg2: 254 -> 244 us per sequence).
    if (P.n_attn + a.units * P.comp_per_unit <= 2 * 148) longer = 0;
    P.n_attn_first = longer * a.units;
    *out = P;
    return true;
}

// Attention with the old cache and the cache update of one chunk in a single launch.
int tensor_chunk_step(lococo_handle* h, const AttnParams& a, const CompressParams& p, cudaStream_t st) {
    TcStepParams P;
    if (!build_step_params(h, a, p, &P)) return -1;
    static bool attr_set[64] = {};
    if (!smem_limit_set(chunk_step_tc_kernel, kMaxSmem, attr_set)) return -1;
    // one CTA per (unit, slot block) and an output cache that is not the input: no partials, no finalize pass
    const bool own_output = p.W_out == nullptr && p.k_out.ptr != p.xk.cache.ptr && p.v_out.ptr != p.xv.cache.ptr;
    P.comp.direct = own_output && P.comp.parts == 1;
    // several CTAs per (unit, slot block): the one that stores the last partial set sums them and writes the rows
    // (the merging CTA stages the stored sets in its idle ring and tiles: every plan has the room, and one that did not
    // would leave the sum to the finalize pass)
    const bool merge_room = (size_t)P.comp.stages * kStageBytes + 4 * 128 * (size_t)P.comp.rows_pad >= 8192 + (size_t)kMergeStage;
    P.comp.merge = own_output && P.comp.parts > 1 && p.R16 == nullptr && merge_room;
    // generation stage: chunks so short that a unit's positions are one small tile. Two units per compress CTA share
    // every weight stage, and a chunk of one query is attended to by a warp instead of a 128-row MMA tile.
    const int n_tile16 = (p.S + 15) / 16 * 16;
    if (own_output && p.R16 == nullptr && p.M == kSlots && p.xk.c == kSlots && p.c_in == kD && p.units > 148 && n_tile16 <= 144 &&
        pair_layout(p.S, n_tile16, p.k).total <= (uint32_t)kMaxSmem && ((P.attn.tma_mask >> kMapVCache) & 1) &&
        (!p.weights_per_head || p.units / p.heads >= 2)) {
        P.comp.pair = 1;
        P.comp.direct = 1;
        P.comp.merge = 0;
        P.comp.n_tile = n_tile16;
        P.comp.tiles = P.comp.parts = P.comp.tiles_per_part = 1;
        P.comp.pairs = p.weights_per_head ? p.heads * ((p.units / p.heads + 1) / 2) : (p.units + 1) / 2;
    }
    int n_attn_ctas = P.n_attn;
    if (a.b == 1 && a.c + 1 <= kDecodeMaxKeys) {
        P.decode = 1;
        P.n_attn_first = 0;
        n_attn_ctas = (a.units + kDecodeUnitsPerCta - 1) / kDecodeUnitsPerCta;
    }
    const int blocks = n_attn_ctas + (P.comp.pair ? P.comp.pairs : a.units * P.comp_per_unit);
    prof_begin(p.prof, 2, st);
    // the step's CTAs read the chunk before they wait for earlier kernels: the first step of a call is therefore
    // launched in plain stream order, after whatever the caller ran before (it may have produced Q, K, V)
    const bool ok = launch_overlapped(chunk_step_tc_kernel, dim3(blocks), dim3(kAttnThreads), kMaxSmem, st, P, h->chain_open) == cudaSuccess;
    h->chain_open = true;
    if (!ok) cudaGetLastError();
    prof_end(p.prof, st);
    if (!ok) return -1;
    if (P.comp.direct || P.comp.merge) return 1;
    const int r = finish_compress(P.comp, st);
    return r < 0 ? -1 : 1 + r;
}

// Whether a chunk step with these parameters can write the new cache straight from its compress CTAs
// (given an output cache that is not the input).
bool tensor_step_direct(lococo_handle* h, const CompressParams& p) {
    Plan pl;
    return h->use_tensor && p.W_out == nullptr && p.R16 == nullptr && make_plan(p.S, p.k, p.c_in / 128, p.units, p.M / kSlots, true, &pl);
}

// ---- persistent chunk loop
static bool sequence_available(lococo_handle* h) {
    if (h->coop_grid == 0) {
        h->coop_grid = -1;
        int dev = 0, sms = 0, per_sm = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return false;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms < 1) return false;
        if (cudaFuncSetAttribute(sequence_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sequence_tc_kernel, kAttnThreads, kMaxSmem) != cudaSuccess ||
            per_sm < 1) {
            cudaGetLastError();
            return false;
        }
        if (cudaHostAlloc(reinterpret_cast<void**>(&h->seq_host),
                          (size_t)lococo_handle::kSeqSlots * kMaxSeqSteps * sizeof(TcStepParams), cudaHostAllocDefault) != cudaSuccess) {
            cudaGetLastError();
            h->seq_host = nullptr;
            return false;
        }
        h->coop_grid = sms * per_sm;
    }
    return h->coop_grid > 0;
}

bool tensor_sequence_add(lococo_handle* h, const AttnParams& a, const CompressParams& p, cudaStream_t st) {
    if (!sequence_available(h) || h->seq_count >= kMaxSeqSteps) return false;
    TcStepParams P;
    if (!build_step_params(h, a, p, &P)) return false;
    P.items_per_unit = P.comp_per_unit + P.qtiles;
    if ((int64_t)h->seq_items + (int64_t)P.items_per_unit * a.units > (int64_t)1 << 30) return false;
    if (h->seq_count == 0) {
        // take the next host slot; make sure the copy that last read it has been carried out
        h->seq_slot = (h->seq_slot + 1) % lococo_handle::kSeqSlots;
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        cudaStreamIsCapturing(st, &cap);
        if (cap == cudaStreamCaptureStatusNone && h->seq_event[h->seq_slot]) cudaEventSynchronize(h->seq_event[h->seq_slot]);
        h->seq_items = 0;
        h->seq_per_unit = 0;
    }
    h->seq_items += P.items_per_unit * a.units;
    h->seq_per_unit += P.items_per_unit;
    P.item_end = h->seq_items;
    P.finished_target = h->seq_per_unit;
    TcStepParams* slot = reinterpret_cast<TcStepParams*>(h->seq_host) + (size_t)h->seq_slot * kMaxSeqSteps;
    slot[h->seq_count++] = P;
    return true;
}

int tensor_sequence_launch(lococo_handle* h, cudaStream_t st, void* prof) {
    const int n = h->seq_count;
    h->seq_count = 0;
    if (n == 0) return 0;
    const TcStepParams* slot = reinterpret_cast<const TcStepParams*>(h->seq_host) + (size_t)h->seq_slot * kMaxSeqSteps;
    TcSeqParams Q{};
    Q.steps = reinterpret_cast<const TcStepParams*>(h->ws + h->off_steps);
    Q.n_steps = n;
    Q.total_items = h->seq_items;
    Q.work = reinterpret_cast<int*>(h->ws + h->off_sync);
    Q.finished = Q.work + 64;
    Q.version = Q.finished + h->units;
    Q.status = reinterpret_cast<int*>(h->ws + h->off_status);
    if (cudaMemcpyAsync(h->ws + h->off_steps, slot, (size_t)n * sizeof(TcStepParams), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemsetAsync(h->ws + h->off_sync, 0, (size_t)(64 + 2 * h->units) * sizeof(int), st) != cudaSuccess)
        return -1;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    cudaStreamIsCapturing(st, &cap);
    if (cap == cudaStreamCaptureStatusNone) {
        if (!h->seq_event[h->seq_slot] && cudaEventCreateWithFlags(&h->seq_event[h->seq_slot], cudaEventDisableTiming) != cudaSuccess)
            return -1;
        cudaEventRecord(h->seq_event[h->seq_slot], st);
    }
    prof_begin(prof, 3, st);
    sequence_tc_kernel<<<std::min(h->coop_grid, Q.total_items), kAttnThreads, kMaxSmem, st>>>(Q);
    const bool ok = cudaGetLastError() == cudaSuccess;
    prof_end(prof, st);
    return ok ? 1 : -1;
}

void tensor_sequence_release(lococo_handle* h) {
    if (h->seq_host) cudaFreeHost(h->seq_host);
    h->seq_host = nullptr;
    for (auto& e : h->seq_event) {
        if (e) cudaEventDestroy(e);
        e = nullptr;
    }
}

bool tensor_attention_supported(const lococo_handle* h, const AttnParams& p) {
    return h->use_tensor && p.d == kD && h->ws != nullptr;
}

int tensor_attention(lococo_handle* h, const AttnParams& p, cudaStream_t st) {
    static bool attr_set[64] = {};
    if (!smem_limit_set(attention_tc_kernel, (int)kAttnSmem, attr_set)) return -1;
    TcAttnParams P{};
    P.base = p;
    P.status = reinterpret_cast<int*>(h->ws + h->off_status);
    fill_attention_maps(&P);
    dim3 grid((p.b + 127) / 128, p.units);
    prof_begin(p.prof, 1, st);
    attention_tc_kernel<<<grid, kAttnThreads, kAttnSmem, st>>>(P);
    const bool ok = cudaGetLastError() == cudaSuccess;
    prof_end(p.prof, st);
    return ok ? 1 : -1;
}

}  // namespace lococo
