// Internal declarations shared by the segkv translation units (host API and kernels).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "segkv.h"

namespace segkv_impl {

constexpr int kMaxCols = 32;       // beams * (heads/kv_heads) handled by one CTA
constexpr int kMaxSplits = 64;     // CTAs that may share one (request, kv head) work group
constexpr int kMaxCluster = 8;     // largest portable thread-block cluster
constexpr int kMaxTiledBeams = 16;  // beams the tiled kernel handles (16 query columns at most)

// {row, mask} pairs.  In the per-request list of DISTINCT response rows `row` indexes the
// response segment's [step*rows + slot] axis; in the per-key record of a response tile in
// shared memory it is the key's step.  `mask` has bit j set when beam j reads the row.
struct URow {
    int32_t row;
    uint32_t mask;
};

// Where and when data was last written: the stream and the per-process sequence number of the launch.
struct WriteMark {
    cudaStream_t stream;
    unsigned long long seq;       // 0: never written
};

struct Dims {
    int batch, beams, heads, kv_heads, head_dim, group;  // group = heads / kv_heads
    int max_prompt, max_steps;
    int rows;                                            // batch * beams
    int chunk_steps;                                     // response capacity grows in chunks of this many steps (0: fixed)
    int dtype;
    int prompt_layout;                                   // SEGKV_PROMPT_HEAD_MAJOR / _TOKEN_MAJOR / _SEQ_FIRST
};

// Element strides of the prompt segment for a request, a kv head and a token in the handle's
// prompt layout (head_dim is always the contiguous dimension).
struct PromptStrides { long long b, h, p; };
inline PromptStrides prompt_strides(const Dims& d) {
    const long long D = d.head_dim, Hkv = d.kv_heads, P = d.max_prompt, B = d.batch;
    switch (d.prompt_layout) {
        case 1: return {P * Hkv * D, D, Hkv * D};        // [B, P, Hkv, D]
        case 2: return {Hkv * D, D, B * Hkv * D};        // [P, B, Hkv, D]
        default: return {Hkv * P * D, P * D, D};         // [B, Hkv, P, D]
    }
}

}  // namespace segkv_impl

struct segkv {
    segkv_impl::Dims d;
    int device;
    int sm_count;
    size_t smem_optin;
    // state
    int prompt_len;      // -1 until segkv_prefill_write
    int steps;
    bool truncated;      // last state change was segkv_truncate_last
    int splits_forced;   // 0 = automatic
    int stages_forced;   // 0 = automatic
    int combine_forced;  // 0 = automatic, 1 = global workspace + ticket, 2 = cluster
    int tile_forced;     // 0 = automatic, 32 or 64 keys per tile of the decode kernel
    int persist_mode;    // -1 = automatic, 0 = never, 1 = always: the persistent form of the separate attention call
    bool overlap;        // programmatic dependent launch between consecutive kernels
    int prefill_groups;  // 0 = automatic; 1 or 2 row groups per CTA of the tcgen05 prefill kernel
    bool fuse_always;    // segkv_decode_step uses the fused kernel even for a single split
    unsigned long long dbg_wait_ns;   // segkv_debug_inject: applies to the next attention launch, then clears
    bool dbg_skip;
    long long launches;
    // device storage (owned)
    void* kp;            // [batch, kv_heads, max_prompt, D] (or the layout chosen by segkv_set_prompt_layout)
    void* vp;
    void* kr;            // [max_steps, rows, kv_heads, D]; K and V of the response segment are ONE
    void* vr;            // allocation (V right behind K), so a V row is its K row plus a constant
    // growing capacity (Section 3.2): chunks of chunk_steps steps, each {K part, V part} in one allocation
    void** k_chunks_host;    // [nchunks_max] device pointers, host copy
    void** k_chunks_dev;     // the same table on the device
    int nchunks, nchunks_max;
    int32_t* parent;     // [max_steps, rows]
    int32_t* anc[2];     // [rows, max_steps], generation t lives in anc[t & 1]
    segkv* leader;       // the handle whose beam-index tables this one uses (segkv_share_index), or NULL
    int followers;       // handles that use THIS one's tables; it cannot be destroyed while there are any
    void* st_pack;       // staging for segkv_step_host_packed: parent | slopes | k | v | q in one block
    cudaEvent_t ev_in, ev_k;   // segkv_layers_step_host: this layer's inputs have arrived / its launch is queued
    void *grp_in, *grp_out;    // segkv_layers_step_host, kept by the first layer of a stack: staging for all of its
    size_t grp_in_cap, grp_out_cap;   // layers in one piece, so that several layers travel in one copy
    int32_t* plens;      // [batch] per-request prompt lengths (segkv_prefill_write_ragged)
    bool ragged;         // plens is in use; prompt_len is then the longest
    segkv_impl::URow* ulist;   // [batch, beams*max_steps] distinct response rows per request
    int32_t* ucount;     // [batch]
    bool lists_valid;    // ulist/ucount describe the newest step (a fused step does not update them)
    // the latest launch that wrote response rows / beam-index tables of this handle, and the one
    // that wrote its row lists (what a later attention launch may read ahead of its wait once
    // these are known to be complete)
    segkv_impl::WriteMark rows_mark, lists_mark;
    int* err_word;       // device error word
    float* ws;           // split workspace
    size_t ws_bytes;
    int* tickets;        // [batch*kv_heads] arrival counters, zero between launches
    int ws_splits;       // splits the workspace was sized for
    // staging for segkv_step_host
    void *st_q, *st_out, *st_k, *st_v;
    int32_t* st_parent;
    float* st_slopes;
    // tensor maps of the prompt segment (valid once prompt_len > 0)
    CUtensorMap tm_kp, tm_vp;
    CUtensorMap tm_kp32, tm_vp32;   // the same arrays in boxes of 32 tokens, for the small-CTA form of the decode kernel
    bool tm_valid;
};

namespace segkv_impl {

// ---- kernels (each returns the cudaError_t of its launch) -----------------
// Rotary embedding applied to the new K rows while they are appended (style 0: none).
struct RopeArgs {
    const float* cos;        // device [positions, D/2]
    const float* sin;
    const int32_t* plens;    // per-request prompt lengths or NULL
    int prompt_len;          // the position of step t's token of request b is prompt length + t
    int style;               // 0 none, SEGKV_ROPE_HALF, SEGKV_ROPE_INTERLEAVED
    int head_dim, kv_heads, bf16;
};

// plens (device, [batch]) or NULL: tokens at or past a request's own length are stored as zeros
cudaError_t launch_prefill_transpose(const Dims& d, const void* k, const void* v, void* kp, void* vp, const int32_t* plens,
                                     int prompt_len, int sm_count, cudaStream_t st);

cudaError_t launch_append(const Dims& d, int step, const int32_t* beam_parent, const void* k_new,
                          const void* v_new, void* kr_slab, void* vr_slab, int32_t* parent_tab,
                          const int32_t* anc_prev, int32_t* anc_cur, URow* ulist, int32_t* ucount,
                          int* err_word, int sm_count, bool pdl, cudaStream_t st, const RopeArgs* rope = nullptr,
                          bool tables = true);
// A read-only pass over `bytes` of device memory (16-byte loads); sink: 64 words of device memory.
cudaError_t launch_read_stream(const void* src, size_t bytes, unsigned* sink, int sm_count, cudaStream_t st);
// Re-derive the distinct-row lists from the current beam-index table (after fused steps).
cudaError_t launch_rebuild_lists(const Dims& d, int steps, const int32_t* anc_cur, URow* ulist, int32_t* ucount,
                                 cudaStream_t st);

struct SdpaArgs {
    const void* q;
    void* out;
    const float* slopes;
    const void* kp;
    const void* vp;
    const void* kr;          // response K (fixed capacity) or NULL (growing: see k_chunks)
    const void* vr;
    const void* const* k_chunks;   // device table of chunk base pointers (growing capacity)
    long long vdelta;        // bytes from a response K row to its V row
    const int32_t* anc;      // beam-index table (fused step: the previous step's)
    const URow* ulist;
    const int32_t* ucount;
    const int32_t* plens;    // device [batch] prompt lengths when they differ per request, else NULL
    float* ws;
    int* tickets;
    int* err_word;
    int prompt_len, steps, splits;
    int tail_groups, tail_splits;   // the last tail_groups work groups get tail_splits splits instead (0: none);
                                    // workspace merge only; the workspace then holds the tail's items when splits == 1
    bool small;              // 32-key tiles and two consumer warps (tensor maps with 32-row boxes)
    bool one_wave;           // every CTA of the launch is resident at once with a few tiles each: latency, not
                             // bandwidth, is what counts; a stage of the ring may be set aside for the response rows
                             // fetched ahead, and what cannot be fetched yet is asked into the L2
    bool cluster;            // merge the splits inside a thread-block cluster
    bool pdl;                // launch with programmatic stream serialisation
    bool prompt_immutable;   // a fully serialised launch has followed the last prompt store
    bool rows_immutable;     // the response rows of earlier steps (separate form: the row lists too) were written by
                             // launches older than this launch's predecessor: readable before the grid-dependency wait
    // fused decode step (append + beam-index update + attention in one launch)
    // test aid (segkv_debug_inject): limit of the kernel's bounded waits (0 = default) and one
    // barrier arrival left out so that a wait runs out
    unsigned long long wait_ns;
    bool dbg_skip;
    bool fused;
    const int32_t* parent;   // [rows] device, NULL at step 0
    const void* k_new;
    const void* v_new;
    void* kr_new_slab;
    void* vr_new_slab;
    int32_t* anc_dst;
    int32_t* parent_row;
};

// Plain gather kernel: one CTA per (beam slot, head), fp32 ALU; kept for shapes
// the tiled kernel does not cover and as an in-library cross-check.
cudaError_t launch_sdpa_rowwise(const Dims& d, const SdpaArgs& a, cudaStream_t st);

// Tiled split-KV kernel (TMA-staged prompt tiles, gathered response rows, tensor-core tiles).
bool tiled_supported(const Dims& d);
bool tiled_cluster_ok(const Dims& d, int splits);        // can `splits` CTAs merge as one cluster?
bool tiled_small_ok(const Dims& d);                      // is there a 32-key-tile form (quarter-SM CTAs) for this shape?
int tiled_tile_keys(int head_dim, bool small);           // rows of one shared-memory tile
size_t tiled_smem_bytes(const Dims& d, int stages, bool small);   // dynamic shared memory of one CTA
// Persistent form of the separate attention call (segkv_sdpa_stream.cu): a resident grid of CTAs walks
// the (work group, split) items round-robin; a.splits items per work group, merged through the workspace.
bool stream_supported(const Dims& d);
int stream_ctas_per_sm();
cudaError_t launch_sdpa_stream(const Dims& d, const SdpaArgs& a, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                               int sm_count, cudaStream_t st);
cudaError_t launch_sdpa_tiled(const Dims& d, const SdpaArgs& a, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                              int stages, cudaStream_t st);

// Same kernel with its split workspace in a fixed device array of the module (no allocation).
size_t tiled_static_scratch_bytes();
cudaError_t launch_sdpa_tiled_static(const Dims& d, SdpaArgs a, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                     int stages, cudaStream_t st, int* too_big);

// Causal prefill attention over the prompt segment.
struct PrefillArgs {
    const void* q;
    void* out;
    const float* slopes;
    int* err_word;
    int prompt_len;
    const CUtensorMap* tm_k;
    const CUtensorMap* tm_v;
    const int32_t* plens;      // device [batch] prompt lengths when they differ per request, else NULL
    // fused prefill: K/V tiles are read from the caller's token-major arrays through these maps and
    // every tile is also stored into the prompt segment (tm_k / tm_v) by one CTA; NULL: read the segment
    const CUtensorMap* tm_k_src;
    const CUtensorMap* tm_v_src;
    const CUtensorMap* tm_q;   // over q as [batch][prompt_len][heads][D], box 64 elements x 128 tokens; NULL if unused
    int row_groups;      // 0 = automatic
    unsigned long long wait_ns;   // test aid, as in SdpaArgs
    bool dbg_skip;
};
// tcgen05 tensor cores with TMEM accumulators; head_dim 64, 128 or 256
bool prefill_tc5_supported(const Dims& d);
cudaError_t launch_prefill_tc5(const Dims& d, const PrefillArgs& a, cudaStream_t st);

}  // namespace segkv_impl
