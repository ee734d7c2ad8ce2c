/*
 * lococo.h - C ABI of the LoCoCo chunk-step library for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-chunk hot path of "LoCoCo: Dropping In
 * Convolutions for Long Context Compression" (arXiv 2406.05317):
 *   Algorithm 2, Step 3   chunk attention over [compressed cache, causal chunk] (Eq. 1)
 *   Algorithm 2, Step 4   mixing logits by a 1-D multi-channel convolution over the
 *                         concatenated [cache; chunk] states (Eq. 6), ReLU
 *                         (Section 3.2.1), sum normalisation (Eq. 7)
 *   Algorithm 2, Step 5   the M cache slots rebuilt as weighted blends of all
 *                         cache and chunk tokens, same weights for K and V (Eq. 4, Eq. 5)
 *   Algorithm 2, loop     attention with the old cache, then fill or compress
 * for batch x heads independent (sequence, head) units.  Notation follows the
 * paper: M cache slots, B chunk size, k conv kernel width, d head dimension.
 *
 * Conventions
 *   - Every pointer named "device" is a CUDA device pointer on the current device,
 *     owned by the caller; the library allocates and frees no device memory and keeps
 *     no pointer after a call returns, except the workspace given to
 *     lococo_set_workspace (which also holds the packed conv weights).
 *   - Tensors are 4-D views [batch, heads, tokens, d] with d contiguous, described by
 *     a lococo_tensor; strides are in elements.  Base pointers and all strides in bytes
 *     must be multiples of 16.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *     enqueue work and return; they do not synchronise unless stated.
 *   - Every entry point returns a lococo_status.  Argument errors are detected on the
 *     host before anything is launched.  Nothing throws, aborts or prints.
 *   - Storage types: LOCOCO_F32 (computed with fp32 FMA) and LOCOCO_BF16 (bf16
 *     operands, fp32 accumulation, fp32 softmax and normalisation).
 */
#ifndef LOCOCO_H_
#define LOCOCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LOCOCO_OK = 0,
    LOCOCO_ERR_INVALID_ARG = 1,       /* NULL / misaligned pointer, bad size, k even, ... */
    LOCOCO_ERR_UNSUPPORTED_SHAPE = 2, /* a shape the kernels do not cover */
    LOCOCO_ERR_WORKSPACE = 3,         /* workspace missing or too small, weights not set */
    LOCOCO_ERR_CUDA = 4,              /* a CUDA runtime call failed */
    LOCOCO_ERR_TIMEOUT = 5            /* a bounded device-side wait ran out */
} lococo_status;

typedef enum { LOCOCO_F32 = 0, LOCOCO_BF16 = 1 } lococo_dtype;

/* Which kernels serve a call. AUTO: tensor-core (tcgen05) kernels where the shape and
 * dtype allow, CUDA-core kernels otherwise. TENSOR_PERSISTENT: the tensor-core kernels, with
 * all consecutive compress steps of a lococo_process_sequence call (Algorithm 2, loop) run by ONE
 * ordinary launch of one CTA per SM instead of one launch per chunk. Its CTAs pull (step, unit,
 * piece) work items from a single list in step order; an item of step n waits (bounded) until the
 * step counter of ITS unit says that the cache of step n-1 is complete, and the CTA that finishes
 * the last item of a (step, unit) pair rebuilds that unit's cache and advances the counter. There
 * is no device-wide barrier and no need for all CTAs to be resident at once: an item only waits
 * for items earlier in the list, which a running CTA has already taken. Results are identical bit
 * for bit to the per-chunk launches. This path is a tested variant, not the default: the per-chunk
 * launches, overlapped as programmatic dependents, are faster at every measured shape. */
typedef enum {
    LOCOCO_PATH_AUTO = 0,
    LOCOCO_PATH_SIMT = 1,
    LOCOCO_PATH_TENSOR = 2,
    LOCOCO_PATH_TENSOR_PERSISTENT = 3
} lococo_path;

typedef struct {
    int32_t batch;            /* sequences processed together */
    int32_t heads;            /* attention heads per sequence */
    int32_t head_dim;         /* d: 64 or 128 */
    int32_t M;                /* cache slots (Section 3.2) */
    int32_t k;                /* conv kernel width, odd (Section 3.2.1; 21 in the paper) */
    int32_t c_in;             /* conv input channels: d (keys) or 2*d (keys stacked on values, Eq. 6) */
    int32_t weights_per_head; /* 0: one weight set [M,c_in,k] shared by the heads (Section 4.1);
                                 1: one set per head [heads,M,c_in,k] */
    int32_t dtype;            /* lococo_dtype of Q, K, V, O, the cache and the weights */
    float softmax_scale;      /* 0 selects 1/sqrt(d) (Eq. 1) */
    float norm_eps;           /* added to the denominator of Eq. 7 */
    int32_t max_chunk;        /* largest chunk length b any call will pass */
    int32_t path;             /* lococo_path */
} lococo_config;

/* Strided view [batch, heads, tokens, d]; element (n,h,t,c) is at
 * ptr + n*stride_batch + h*stride_head + t*stride_token + c (in elements). */
typedef struct {
    void* ptr; /* device */
    int64_t stride_batch, stride_head, stride_token;
} lococo_tensor;

typedef struct lococo_handle lococo_handle;

/* Validates the configuration and returns a host-side handle. No device work. */
lococo_status lococo_create(const lococo_config* config, lococo_handle** out);
lococo_status lococo_destroy(lococo_handle* handle);

/* Bytes of device scratch the handle needs (packed weights, mixing logits, partial
 * blends, status word). */
lococo_status lococo_workspace_bytes(const lococo_handle* handle, size_t* out);
/* Gives the handle its scratch: device memory, 256-byte aligned, at least
 * lococo_workspace_bytes; it must stay valid until lococo_destroy or the next
 * lococo_set_workspace.  Clears the device status word on `stream`. */
lococo_status lococo_set_workspace(lococo_handle* handle, void* device_ptr, size_t bytes, void* stream);

/* Conv weights of Eq. 6: G [heads|1, M, c_in, k] and optional bias [heads|1, M]
 * (NULL = none), device pointers in the configured dtype, contiguous.  They are
 * re-packed into the workspace, so the workspace must be set first and G may be
 * released after the stream reaches this point. */
lococo_status lococo_set_weights(lococo_handle* handle, const void* G_device, const void* bias_device,
                                 void* stream);

/* Protected slots (Section 5.2, Table 6: the compressor next to an eviction policy that always
 * keeps some tokens, such as the initial "sink" tokens).  The paper gives no formula; this
 * library's reading: for the first `slots` cache slots the row of Eq. 7's weight matrix is the
 * unit row e_i, so slot i keeps entry i of [cache; chunk] bit for bit (after the fill steps:
 * token i of the sequence), the convolution still reads every entry, the other slots are
 * compressed as before, and no gradient reaches the conv weights of those rows.
 * 0 <= slots <= M; 0 (the default) is the plain method.  Host-side state only: it applies to
 * every later compress step, chunk loop and backward pass of this handle. */
lococo_status lococo_set_protected_slots(lococo_handle* handle, int32_t slots);

/*
 * Algorithm 2, the branch after Step 3.  With c = cache_len:
 *   c + b <= M : fill - chunk rows are appended at cache rows c..c+b-1;
 *   otherwise  : Steps 4 and 5 on the S = c + b real entries [cache; chunk]:
 *       A[i,j] = bias_i + sum_ch sum_t G[i,ch,t] * Z[j+t-(k-1)/2, ch]   (zero outside [0,S))
 *       R = max(A, 0);  s_i = sum_j R[i,j] + eps;  w = R / s              (Eq. 7)
 *       K_out[i,:] = sum_j w[i,j] XK[j,:];  V_out likewise                (Eq. 4, Eq. 5)
 *     with Z = XK (c_in = d) or [XK | XV] along channels (c_in = 2d).
 * K_cache/V_cache hold M rows per unit of which the first c are valid; the outputs
 * may alias them.  new_cache_len (host, optional) receives c + b or M.
 * W_out (device, optional, fp32 [batch, heads, M, c+b]) receives w of a compress step.
 */
lococo_status lococo_compress_step(lococo_handle* handle, lococo_tensor K_cache, lococo_tensor V_cache,
                                   int32_t cache_len, lococo_tensor K_chunk, lococo_tensor V_chunk, int32_t b,
                                   lococo_tensor K_cache_out, lococo_tensor V_cache_out,
                                   int32_t* new_cache_len, float* W_out, void* stream);

/*
 * The compress branch of lococo_compress_step for callers that cannot allocate device
 * memory at all.  (The paper has no counterpart of this entry point; it computes exactly
 * Steps 4 and 5 of Algorithm 2 as described above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plugin inside a host
 * application that owns every byte of device memory and hands out none, a process whose
 * memory pool was sized up front and is full, or a latency-critical loop in which an
 * allocation (a synchronising driver call) is not acceptable.  Such a caller cannot provide
 * the workspace lococo_set_workspace asks for.  Here the scratch (packed weights, mixing
 * logits, row sums, partial blends) sits in a fixed 8 MiB array compiled into the library,
 * which every GPU that loads the library keeps resident until the process exits.  No
 * handle is needed and nothing is allocated or freed, on the host or on the device.
 *
 * cfg describes the problem as for lococo_create (max_chunk, path and softmax_scale are
 * ignored); G [heads|1, M, c_in, k] and bias (or NULL) are device pointers in cfg->dtype and
 * are re-packed on every call.  The tensors are those of lococo_compress_step; the outputs may
 * be the cache inputs themselves (same base pointer and strides: an update in place).  As in
 * lococo_compress_step only equal base pointers are recognised: an output that overlaps another
 * tensor at an offset is not detected and gives undefined results.
 * Only a real compress step is accepted (cache_len + b > M): the fill
 * branch needs no scratch, use lococo_compress_step for it.
 * Errors: LOCOCO_ERR_WORKSPACE when the scratch this problem needs, about
 *   4*batch*heads*M*(cache_len+b) + 8*batch*heads*M*d + sizeof(G) bytes,
 * exceeds the built-in limit (lococo_static_scratch_limit); LOCOCO_ERR_INVALID_ARG /
 * LOCOCO_ERR_UNSUPPORTED_SHAPE as for the other calls, before anything is launched.
 * The first call on each device looks up the device address of the array (a runtime
 * query); make that call outside any stream capture.  All calls on a device share the one
 * array: every byte a call reads it has written first, so nothing needs clearing between
 * calls, but two calls whose kernels overlap on the GPU (different streams, no dependency)
 * race on it - order them.
 */
lococo_status lococo_compress_step_static(const lococo_config* cfg, const void* G_device, const void* bias_device,
                                          lococo_tensor K_cache, lococo_tensor V_cache, int32_t cache_len,
                                          lococo_tensor K_chunk, lococo_tensor V_chunk, int32_t b,
                                          lococo_tensor K_cache_out, lococo_tensor V_cache_out, void* stream);
/* Size in bytes of the built-in scratch array used by lococo_compress_step_static. */
lococo_status lococo_static_scratch_limit(size_t* out);

/*
 * Algorithm 2, Step 3 (Eq. 1): the b chunk queries attend over the c cache entries
 * (all visible) followed by the chunk (query r sees chunk keys 0..r), softmax over
 * keys with scale softmax_scale.  lse (device, optional, fp32 [batch, heads, b])
 * receives the log-sum-exp of the scaled logits.
 */
lococo_status lococo_chunk_attention(lococo_handle* handle, lococo_tensor Q_chunk, lococo_tensor K_cache,
                                     lococo_tensor V_cache, int32_t cache_len, lococo_tensor K_chunk,
                                     lococo_tensor V_chunk, int32_t b, lococo_tensor O_chunk, float* lse,
                                     void* stream);

/* Bytes of the `saved` buffer lococo_process_sequence fills for a later backward pass:
 * the cache before every step, and the attention log-sum-exp. */
lococo_status lococo_saved_bytes(const lococo_handle* handle, int32_t L, int32_t B, size_t* out);

/*
 * Algorithm 2 over L tokens in chunks of B (the last chunk may be short): for each
 * chunk, lococo_chunk_attention with the cache as it stands, then lococo_compress_step.
 * Q, K, V, O hold L tokens; K_cache/V_cache (M rows per unit) and *cache_len_inout
 * (host) carry the cache state in and out, so a sequence can be suspended and resumed
 * between calls.  saved (device, optional) is laid out as lococo_saved_bytes describes.
 * Calls that repeat the previous call's arguments exactly (same views, L, B, cache length) on a
 * capturable stream (not the legacy default stream) are replayed from a cached CUDA graph from the
 * third such call on; buffer contents may change freely between calls.
 */
lococo_status lococo_process_sequence(lococo_handle* handle, lococo_tensor Q, lococo_tensor K, lococo_tensor V,
                                      int32_t L, int32_t B, lococo_tensor O, lococo_tensor K_cache,
                                      lococo_tensor V_cache, int32_t* cache_len_inout, void* saved, void* stream);

/* Bytes of device staging lococo_process_sequence_host needs for L tokens. */
lococo_status lococo_host_staging_bytes(const lococo_handle* handle, int32_t L, size_t* out);

/*
 * lococo_process_sequence on HOST buffers: contiguous [batch, heads, L, d] Q, K, V are
 * copied to the device staging area, the loop runs from an empty cache, and O plus the
 * final cache ([batch, heads, M, d] each, optional) are copied back.  The three legs are
 * pipelined chunk by chunk on streams the handle owns (inputs of chunk n+1, the step of
 * chunk n, the output of chunk n-1), ordered after the work already queued on `stream`.
 * Host buffers should be pinned for the copies to be asynchronous.  Synchronises `stream`
 * before returning; final_cache_len (host) receives the fill count.
 */
lococo_status lococo_process_sequence_host(lococo_handle* handle, const void* Q_host, const void* K_host,
                                           const void* V_host, int32_t L, int32_t B, void* O_host,
                                           void* K_cache_host, void* V_cache_host, int32_t* final_cache_len,
                                           void* device_staging, size_t staging_bytes, void* stream);

/*
 * Gradients of  loss = <dO, O> + <dK_cache_final, K_cache_final> + <dV_cache_final, V_cache_final>
 * through one lococo_process_sequence call (the training use of Algorithm 2; Section 3.2.1: the
 * conv parameters are trained end to end).
 * Q, K, V, O: the forward's tensors; cache_len_in: the cache fill count that forward started from
 * (0: an empty cache); saved: what that forward wrote (it holds the cache before every step).
 * dQ, dK, dV (configured dtype) are overwritten; dG (fp32 [heads|1, M, c_in, k]) and
 * dbias (fp32 [heads|1, M], optional) are accumulated (+=), summed over the units that
 * share a weight set.  dK_cache_final/dV_cache_final may have ptr == NULL (zero).
 * dK_cache_in/dV_cache_in ([batch, heads, M, d], configured dtype, ptr == NULL: not wanted) receive
 * the gradient w.r.t. the cache the forward started from (rows at and beyond cache_len_in: zeros).
 * A sequence processed in several forward calls is differentiated call by call, last call first,
 * each call's dK_cache_in/dV_cache_in being the dK_cache_final/dV_cache_final of the call before it.
 * scratch: device memory of lococo_backward_scratch_bytes.
 */
lococo_status lococo_backward_scratch_bytes(const lococo_handle* handle, int32_t L, int32_t B, size_t* out);
lococo_status lococo_process_sequence_backward(lococo_handle* handle, lococo_tensor Q, lococo_tensor K,
                                               lococo_tensor V, lococo_tensor O, int32_t L, int32_t B,
                                               int32_t cache_len_in, const void* saved, lococo_tensor dO,
                                               lococo_tensor dK_cache_final, lococo_tensor dV_cache_final,
                                               lococo_tensor dQ, lococo_tensor dK, lococo_tensor dV, float* dG,
                                               float* dbias, lococo_tensor dK_cache_in, lococo_tensor dV_cache_in,
                                               void* scratch, size_t scratch_bytes, void* stream);

/* Synchronises `stream` and reads the device status word: LOCOCO_OK, or
 * LOCOCO_ERR_TIMEOUT if a bounded wait inside a kernel gave up (results invalid).  The word
 * stays set, and the workspace's internal counters may be left mid-step, until the workspace
 * is handed over again with lococo_set_workspace (followed by lococo_set_weights). */
lococo_status lococo_get_last_device_status(lococo_handle* handle, int32_t* out, void* stream);

/* Number of kernels this handle has launched so far (host-side counter). */
lococo_status lococo_launch_count(const lococo_handle* handle, int64_t* out);

/*
 * Optional timing of single kernel classes with CUDA events recorded on the launching
 * stream around each launch.  kind 0: the kernel that evaluates Eq. 6 (the conv
 * contraction, with whatever is fused into it); kind 1: the chunk-attention kernel (Eq. 1);
 * kind 2: the single launch lococo_process_sequence uses per chunk on the tensor-core path, which
 * holds both of the above (Step 3 and Steps 4-5 of Algorithm 2 are independent of each other);
 * kind 3: the persistent launch that runs all consecutive compress steps of a lococo_process_sequence call.
 * lococo_profile_enable(h, 1) starts a fresh recording, (h, 0) stops it;
 * lococo_profile_read waits for the recorded events and returns the summed duration in
 * milliseconds and the number of launches of that kind since the recording started.
 */
lococo_status lococo_profile_enable(lococo_handle* handle, int32_t on);
lococo_status lococo_profile_read(lococo_handle* handle, int32_t kind, double* total_ms, int64_t* launches);

const char* lococo_status_string(lococo_status status);

#ifdef __cplusplus
}
#endif
#endif /* LOCOCO_H_ */
