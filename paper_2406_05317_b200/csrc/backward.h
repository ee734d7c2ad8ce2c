// Shared by the CUDA-core and the tensor-core backward kernels.
#pragma once
#include "common.cuh"

struct lococo_handle;

namespace lococo {

// One reversed step of Algorithm 2 for all units.
struct BwdStep {
    CatView xk, xv;            // [saved cache; chunk]
    View q, o, d_o;            // this chunk's queries, outputs, output gradients
    View dq, dk, dv;           // this chunk's gradients (outputs)
    int heads, units, d, M, k, c_in, c, b, S;
    int weights_per_head;
    const void* g_packed;      // [sets][k][M][c_in]
    float scale;
    const float* lse;          // this chunk's log-sum-exp, [units][lse_stride]
    int64_t lse_stride;
    float *R, *s;              // recomputed ReLU'd logits [units][M][S] and denominators [units][M]
    float* dA;                 // [units][M][S]: dw, then dA in place
    float* delta;              // [units][b]: <dO_r, O_r>
    float *gK, *gV;            // [units][M][d] gradient w.r.t. the cache (after the step in, before the step out)
    float *dXK, *dXV;          // [units][S][d]
    float *dG, *dbias;         // [sets][M][c_in][k], [sets][M]
};

// Tensor-core versions of the step's contractions (bf16, d = 128, M a multiple of 128). The scratch is
// carved from the caller's backward scratch; every function returns the number of launches or -1.
bool tensor_backward_supported(const lococo_handle* h);
size_t tensor_backward_scratch_bytes(const lococo_handle* h, int B);
int tensor_backward_prepare(lococo_handle* h, int B, char* scratch, cudaStream_t st);
int tensor_backward_pack(lococo_handle* h, const BwdStep& p, int B, char* scratch, cudaStream_t st);
int tensor_backward_compress(lococo_handle* h, const BwdStep& p, const CompressParams& fwd, int B, char* scratch, cudaStream_t st);
int tensor_backward_attention(lococo_handle* h, const BwdStep& p, int B, char* scratch, cudaStream_t st);

}  // namespace lococo
