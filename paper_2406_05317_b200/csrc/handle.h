// Host-side state behind a lococo_handle, and the hooks of the tensor-core path.
#pragma once

#include <vector>

#include "common.cuh"

namespace lococo {
// Optional CUDA-event timing of individual kernel classes, on the launching stream.
enum ProfKind { PROF_CONV = 0, PROF_ATTENTION = 1, PROF_STEP = 2, PROF_SEQUENCE = 3, PROF_KINDS = 4 };
struct Profiler {
    struct Rec { cudaEvent_t a, b; int kind; };
    bool on = false;
    std::vector<Rec> recs;  // event pairs, reused across profile runs
    size_t used = 0;
    void begin(int kind, cudaStream_t st);
    void end(cudaStream_t st);
    void release();
};
}  // namespace lococo

struct lococo_handle {
    lococo_config cfg{};
    int prot = 0;   // protected slots (Section 5.2)
    int units = 0;          // batch * heads
    size_t elt = 0;         // bytes per stored element
    float scale = 0.f;      // softmax scale in effect
    bool use_tensor = false;
    // true once a kernel of this library has been launched in the current call: only then may the next one be
    // launched as a programmatic dependent (its early, pre-wait reads must not race with a foreign kernel)
    bool chain_open = false;
    bool persistent_loop = false;   // consecutive compress steps as one persistent launch (LOCOCO_PATH_TENSOR_PERSISTENT)
    bool weights_set = false;
    bool has_bias = false;
    char* ws = nullptr;     // caller-owned device workspace
    size_t ws_need = 0;
    size_t off_status = 0, off_gpack = 0, off_bias = 0, off_s = 0, off_UK = 0, off_UV = 0, off_R = 0;
    size_t off_gimage = 0, off_part = 0, off_steps = 0, off_sync = 0;  // tensor-core path
    size_t off_alt_k = 0, off_alt_v = 0;   // second cache (the chunk loop alternates between the caller's and this one)
    size_t off_merge = 0;                  // per (unit, slot block): partial sets stored in the current step
    // persistent chunk loop: step descriptors staged in pinned host memory (a small ring, one slot per call)
    static constexpr int kSeqSlots = 4;
    unsigned char* seq_host = nullptr;
    cudaEvent_t seq_event[kSeqSlots] = {};
    int seq_slot = 0, seq_count = 0;
    // lococo_process_sequence_host: copy streams and per-chunk events (created on first use)
    cudaStream_t host_in = nullptr, host_out = nullptr;
    cudaEvent_t* host_ev = nullptr;
    int host_ev_n = 0;
    int seq_items = 0, seq_per_unit = 0;   // items queued so far: all units, one unit
    int coop_grid = 0;      // 0: not probed yet, -1: persistent kernel unavailable, > 0: CTAs that fit the device
    int64_t launches = 0;
    // CUDA graph of the chunk loop for the most recent argument set of lococo_process_sequence
    struct LoopGraph {
        unsigned char key[256] = {};   // the call's arguments, byte for byte
        size_t key_len = 0;
        int seen = 0;                  // identical calls so far (the graph is captured on the second)
        cudaGraphExec_t exec = nullptr;
        int64_t launches = 0;          // kernels inside the graph
        int c_out = 0;                 // cache length after the loop
        bool disabled = false;         // a graph call failed once: stay eager
    } loop_graph;
    lococo::Profiler prof;
};

namespace lococo {

// Tensor-core (tcgen05) path, tensor_forward.cu.
bool tensor_config_supported(const lococo_config* c);
void tensor_layout_workspace(lococo_handle* h, size_t* off);
int tensor_pack_weights(lococo_handle* h, const void* G, cudaStream_t st);
bool tensor_compress_supported(const lococo_handle* h, const CompressParams& p);
int tensor_compress(lococo_handle* h, const CompressParams& p, cudaStream_t st);
bool tensor_step_direct(lococo_handle* h, const CompressParams& p);
bool tensor_attention_supported(const lococo_handle* h, const AttnParams& p);
int tensor_attention(lococo_handle* h, const AttnParams& p, cudaStream_t st);
int tensor_chunk_step(lococo_handle* h, const AttnParams& a, const CompressParams& p, cudaStream_t st);
// Persistent chunk loop: queue consecutive compress steps, then run them all in one launch of one CTA per SM.
bool tensor_sequence_add(lococo_handle* h, const AttnParams& a, const CompressParams& p, cudaStream_t st);
int tensor_sequence_launch(lococo_handle* h, cudaStream_t st, void* prof);
void tensor_sequence_release(lococo_handle* h);

}  // namespace lococo
