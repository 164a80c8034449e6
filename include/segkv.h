/*
 * segkv — decode-step attention over a segment KV cache, for NVIDIA B200 (sm_100a).
 *
 * One handle is one attention layer's cache.  The cache has two segments
 * (paper Section 3.2, "Segment KV Cache"):
 *   - the PROMPT segment: K/V of each request's prompt, stored once per request
 *     and shared by all of its beams;
 *   - the RESPONSE segment: K/V of generated tokens, sequence-first
 *     [step, batch*beams, kv_heads, head_dim] (Section 3.1), written in place,
 *     one slab per decode step, never concatenated or re-ordered.
 * Beam search hands over, per step, which earlier beam each beam slot extends.
 * Instead of re-ordering the past cache with an index select (Section 3.1,
 * Fig. 1) the library keeps those parent ids, derives the beam-index table
 * (Section 3.3, "Index select fusion") and lets the attention kernel read the
 * response rows through it.
 *
 * Conventions for every entry point
 *   - return value: SEGKV_OK (0) or a negative SEGKV_E* code; no exceptions, no
 *     process exit, no device-side trap;
 *   - "device pointer" = memory of the device that was current at segkv_create,
 *     16-byte aligned, contiguous in the stated layout, owned by the caller and
 *     only read/written by the work the call enqueues;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream); calls that enqueue work are asynchronous on it;
 *   - the handle is not thread-safe; calls on one handle must be ordered by
 *     the caller (same stream, or explicit synchronisation);
 *   - beam slot g = b*beams + j (request b, beam j); query head h reads kv head
 *     h / (heads/kv_heads).
 */
#ifndef SEGKV_H
#define SEGKV_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SEGKV_API __attribute__((visibility("default")))
#else
#define SEGKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct segkv* segkv_t;

enum { SEGKV_F16 = 0, SEGKV_BF16 = 1 };

enum {
    SEGKV_OK = 0,
    SEGKV_EINVAL = -1,    /* bad dimension, NULL/unaligned pointer, unknown dtype        */
    SEGKV_ESTATE = -2,    /* call out of order (append before prefill, wrong step, ...)  */
    SEGKV_ECAPACITY = -3, /* prompt_len > max_prompt or step >= max_steps                */
    SEGKV_ENOMEM = -4,    /* host or device allocation failed                            */
    SEGKV_ECUDA = -5,     /* a CUDA call failed; segkv_last_cuda_error() names it        */
    SEGKV_EDEVICE = -6    /* a kernel reported a problem; see segkv_get_error()          */
};

/* bits of the device error word returned by segkv_get_error */
enum {
    SEGKV_DEV_BAD_PARENT = 1, /* a beam_parent value outside [0,beams) was clamped       */
    SEGKV_DEV_WAIT_LIMIT = 2  /* a bounded wait inside a kernel ran out (never expected) */
};

/*
 * Allocate one layer's cache on the current device: prompt segment
 * [batch, kv_heads, max_prompt, head_dim] x {K,V}, response segment
 * [max_steps, batch*beams, kv_heads, head_dim] x {K,V} (pre-allocated to
 * max_steps, the fixed-capacity variant Section 3.2 describes), the parent
 * table [max_steps, batch*beams], the beam-index tables and the split
 * workspace of the attention kernel.
 * Requirements: all dims > 0 (max_prompt may be 0), heads % kv_heads == 0,
 * head_dim in {64,128,256}, beams*(heads/kv_heads) <= 32, dtype SEGKV_F16/BF16.
 * The softmax scale is 1/sqrt(head_dim).
 * Errors: EINVAL, ENOMEM, ECUDA.  *out is set only on success.
 */
SEGKV_API int segkv_create(segkv_t* out, int batch, int beams, int heads, int kv_heads, int head_dim,
                 int max_prompt, int max_steps, int dtype);

/*
 * Like segkv_create, but the response segment grows with the response
 * (Section 3.2: N_step is raised in steps of 16 so that short responses do not
 * pay for the model's maximum length): storage for `chunk_steps` more steps is
 * allocated when step chunk_steps, 2*chunk_steps, ... is appended, and the K/V
 * held after n steps follow Eq. 3 with step = chunk_steps.  Unlike the paper's
 * scheme nothing is copied or freed when the capacity grows: the chunks are
 * separate allocations that the kernels address through a small table.
 * max_steps stays the upper bound (it sizes the index tables).  chunk_steps 0,
 * or >= max_steps, is segkv_create.  The append / decode-step call that opens
 * a chunk calls cudaMalloc.  Errors: as segkv_create.
 */
SEGKV_API int segkv_create_growing(segkv_t* out, int batch, int beams, int heads, int kv_heads, int head_dim,
                                   int max_prompt, int max_steps, int chunk_steps, int dtype);

/* K/V bytes the handle holds right now: batch * (max_prompt + beams * steps held) * 2*kv_heads*head_dim*2
 * (Eq. 3 for one layer; "steps held" is max_steps, or the chunks opened so far). */
SEGKV_API long long segkv_allocated_kv_bytes(segkv_t h);

/* Free everything the handle owns.  Synchronises the device.  NULL is allowed.
 * ESTATE (and nothing freed) while other handles use this one's tables
 * (segkv_share_index). */
SEGKV_API int segkv_destroy(segkv_t h);

/*
 * Store the prompt K/V (Section 3.2: kept once per request at prefill).
 * k, v: device pointers, token-major [batch, prompt_len, kv_heads, head_dim],
 * the layout a fused QKV projection produces (Section 3.1 batch-first).  The
 * library keeps them head-major [batch, kv_heads, prompt_len, head_dim].
 * Resets the number of appended steps to 0.  prompt_len == 0 is allowed (then
 * k and v may be NULL).  Errors: EINVAL, ECAPACITY, ECUDA.
 */
SEGKV_API int segkv_prefill_write(segkv_t h, const void* k, const void* v, int prompt_len, void* stream);

/*
 * The same for prompts of different lengths (the paper's experiments use one
 * prompt length per batch; a serving batch does not).  k, v: device, token-major
 * [batch, padded_len, kv_heads, head_dim], request b's tokens in rows
 * [0, prompt_lens[b]) and anything at all in the padding behind them.
 * prompt_lens: HOST int32 [batch], each in [1, padded_len]; copied before the
 * call returns.  Every later call on the handle then uses request b's own
 * length: the decode attention and the fused step attend to its prompt_lens[b]
 * prompt tokens followed by the response steps, ALiBi positions count from its
 * own length.  The padding is stored as zeros.  segkv_prompt_len returns
 * padded_len.  segkv_prefill_sdpa takes q and out in the padded shape, computes
 * rows [0, prompt_lens[b]) of request b and leaves the rows behind them in out
 * untouched.  A later segkv_prefill_write returns the handle to one length.
 * Errors: EINVAL (NULL, a length out of range), ECAPACITY, ECUDA.
 */
SEGKV_API int segkv_prefill_write_ragged(segkv_t h, const void* k, const void* v, int padded_len,
                                         const int32_t* prompt_lens, void* stream);

/*
 * Prefill attention (Section 3.1: at prefill Query_0/Key_0/Value_0 arrive batch-first and the
 * customised SDPA kernel takes and returns that layout; Section 3.3: it is the special case of
 * the decode kernel that sees only query and prompt key/value).  Causal self-attention of every
 * prompt position over the positions up to itself, K/V read from the prompt segment that
 * segkv_prefill_write has stored:
 *     out[b,i,hd,:] = softmax_{j<=i}(q[b,i,hd,:] . K[b,j,:] / sqrt(head_dim) + bias) . V[b,j,:]
 *   q, out: device [batch, prompt_len, heads, head_dim] (token-major, like k and v of the write);
 *   alibi_slopes: device float [heads] or NULL; bias = slope[hd] * (j - i).
 * fp16/bf16 operands, fp32 scores/softmax/accumulation, output rounded to nearest-even.
 * Errors: EINVAL, ESTATE (no prompt stored), ECUDA.
 *
 * segkv_prefill does what segkv_prefill_write followed by segkv_prefill_sdpa does, in ONE launch:
 * the attention kernel reads K/V from the caller's k and v (as given to segkv_prefill_write) and
 * stores every tile into the prompt segment on its way through shared memory, each tile by exactly
 * one CTA, so no separate copy of the prompt is made first.  The segment and the output agree bit
 * for bit with the two-call form.  Errors: those of the two calls.
 */
SEGKV_API int segkv_prefill_sdpa(segkv_t h, const void* q, void* out, const float* alibi_slopes, void* stream);
SEGKV_API int segkv_prefill(segkv_t h, const void* k, const void* v, const void* q, void* out, int prompt_len,
                            const float* alibi_slopes, void* stream);

/*
 * Decode step `step` (0-based), before its attention call: write the step's
 * new K/V rows into slab `step` of the response segment (Section 3.1: Key_t,
 * Value_t kept in place in the pre-allocated buffer), record the beam parents
 * as row `step` of the parent table, and update the beam-index table
 * (Section 3.3) so that it resolves every beam slot's row at every step <= step.
 *   beam_parent: device int32 [batch*beams]; value = LOCAL beam id in [0,beams)
 *                of the slot (same request) at step-1 that this slot extends.
 *                Ignored, and may be NULL, when step == 0: all beams descend
 *                from the shared prompt.  Out-of-range values are clamped into
 *                range and flagged in the device error word (SEGKV_DEV_BAD_PARENT).
 *   k_new, v_new: device [batch*beams, kv_heads, head_dim].
 * `step` must equal the number of steps appended so far.
 * Errors: EINVAL, ESTATE (no prefill yet, wrong step), ECAPACITY, ECUDA.
 */
SEGKV_API int segkv_append(segkv_t h, int step, const int32_t* beam_parent, const void* k_new,
                 const void* v_new, void* stream);

/*
 * The fused decode attention (Section 3.3, "Customized SDPA Kernel"): for every
 * beam slot g and head hd,
 *     out[g,hd,:] = softmax(q[g,hd,:] . K^T / sqrt(head_dim) + bias) . V
 * over the request's prompt rows followed by the beam's own response row of
 * every appended step, selected through the beam-index table inside the kernel.
 * fp16/bf16 operands, fp32 scores, softmax and accumulation, output rounded to
 * nearest-even in the cache dtype.
 *   q, out: device [batch*beams, heads, head_dim] (Section 3.3: [1, BSxBW, H, D]).
 *   alibi_slopes: device float [heads] or NULL.  When given, bias for the key
 *       at sequence position p is slope[hd] * (p - qpos), prompt rows at
 *       p = 0..prompt_len-1, the step-s row at prompt_len + s, qpos the newest
 *       position.  (ALiBi is not in the paper; the Bloom workload needs it.)
 * With no step appended the call attends to the prompt only (the paper's
 * "special case" of the kernel).  The call may be repeated; it changes nothing
 * but `out` and the library's own workspace.
 * Errors: EINVAL, ESTATE (nothing to attend to), ECUDA.
 */
SEGKV_API int segkv_decode_sdpa(segkv_t h, const void* q, void* out, const float* alibi_slopes, void* stream);

/*
 * One decode step in ONE launch: exactly segkv_append(step, ...) followed by
 * segkv_decode_sdpa(q, out, ...), fused (Section 3.1-3.3 taken together: the
 * step's Key_t/Value_t, its beam indices and the attention over prompt +
 * responses).  The attention kernel derives the new beam-index column from
 * `beam_parent` and the previous step's table while it gathers, reads the new
 * rows straight from k_new / v_new, and stores rows, parents and table for the
 * following steps.  Saves a launch and a dependent memory round trip per layer.
 * Arguments, layouts and errors are those of the two calls.  The library runs
 * the step as the two launches instead where that is the faster form or the only
 * one: shapes with more than 16 query columns per kv head, handles that share
 * another handle's tables, launches whose work groups fill the GPU without being
 * split, and launches whose CTAs would each have many steps' rows or many prompt
 * tiles to go through.  Both forms give the same beam-index tables bit by bit and
 * outputs within the stated tolerance of each other (the rows are visited in a
 * different order).
 */
SEGKV_API int segkv_decode_step(segkv_t h, int step, const int32_t* beam_parent, const void* k_new,
                                const void* v_new, const void* q, void* out, const float* alibi_slopes,
                                void* stream);

/*
 * segkv_decode_sdpa for callers that must not allocate device memory.  (The
 * paper has no counterpart: this is a deployment variant of the same kernel.)
 *
 * Who needs it: segkv_decode_sdpa keeps its split workspace in memory the handle
 * allocates with cudaMalloc (at create time, and again when segkv_set_tuning
 * asks for more splits than that covers).  A caller inside a serving loop whose memory
 * pool owns the whole device, a caller whose next request must not stall
 * behind the device-wide synchronisation an allocation implies, or a caller
 * that is not allowed to call the CUDA allocator at all (a plug-in running
 * under someone else's allocator policy) cannot afford that.  This entry point
 * calls no allocator: the partial outputs of the splits, their max/sum pairs
 * and the arrival counters of the workspace merge live in an 8 MiB array that
 * is part of the library image; every GPU that loads the library holds those
 * 8 MiB until the process exits.
 *
 * Arguments, results and errors are those of segkv_decode_sdpa; the output
 * agrees with it within the path's tolerance (the splits are always merged
 * through the workspace, never inside a cluster, so the summation order can
 * differ).  In addition:
 *   - ECAPACITY when batch*kv_heads*splits*beams*(heads/kv_heads)*(head_dim+2)
 *     floats plus the counters exceed the 8 MiB (segkv_last_cuda_error() says
 *     so); nothing is launched then.  Fewer splits (segkv_set_tuning) shrink
 *     the need; one split needs none.  EINVAL for shapes with more than 16
 *     query columns per kv head, which the tiled kernel does not take;
 *   - the first call on each device looks the array's device address up
 *     (cudaGetSymbolAddress, with the handle's device current).  Make that
 *     first call before any stream capture begins, and from one host thread
 *     (later calls only read the stored address);
 *   - all handles and all calls share the one array, and it keeps what the
 *     last call left: the counters are cleared on the stream at the start of
 *     every call, and two calls that overlap on the GPU (different streams, or
 *     this and another handle) corrupt each other's partials.  Order them.
 */
SEGKV_API int segkv_decode_sdpa_static(segkv_t h, const void* q, void* out, const float* alibi_slopes,
                                       void* stream);

/*
 * One whole decode step from HOST memory: copies beam_parent, k_new, v_new, q
 * (and slopes, if given) to the device, runs segkv_decode_step,
 * copies `out` back and waits for it.  All pointers are host pointers (pinned
 * memory makes the copies asynchronous); layouts as in the device calls.
 * Staging buffers are part of the handle.  Errors: as the two calls.
 */
SEGKV_API int segkv_step_host(segkv_t h, int step, const int32_t* beam_parent, const void* k_new,
                    const void* v_new, const void* q, void* out, const float* alibi_slopes,
                    void* stream);

/*
 * segkv_step_host with the step's inputs packed into ONE host block, so that a step
 * costs one copy in, one launch and one copy out (each cudaMemcpyAsync costs
 * several microseconds, more than the kernel at small shapes).
 * segkv_host_pack_bytes returns the size of the block and, if `offsets` is not
 * NULL, the byte offsets of its five sections in offsets[0..4]: beam_parent
 * (int32 [rows]), alibi slopes (float [heads]), k_new, v_new, q (layouts as in
 * segkv_decode_step); every section starts on a 256-byte boundary.  host_in is
 * that block (the parent section is ignored at step 0, the slopes section when
 * has_slopes == 0), host_out receives `out`.  Both are host pointers, pinned
 * for asynchronous copies.  Errors: as segkv_step_host.
 */
SEGKV_API size_t segkv_host_pack_bytes(segkv_t h, size_t* offsets);
SEGKV_API int segkv_step_host_packed(segkv_t h, int step, const void* host_in, void* host_out, int has_slopes,
                                     void* stream);

/*
 * segkv_step_host_packed without the wait at the end: the copy in, the launch and
 * the copy out are queued on `stream` and the call returns.  The caller waits for
 * the stream (or an event behind the call) before reading host_out or reusing
 * host_in; a model that drives its layers from host buffers waits once per step,
 * not once per layer, and the queue of one layer overlaps the host work of the
 * next.  No counterpart in the paper (an interface convenience).  Errors: as
 * segkv_step_host_packed.
 */
SEGKV_API int segkv_step_host_packed_async(segkv_t h, int step, const void* host_in, void* host_out, int has_slopes,
                                 void* stream);

/*
 * segkv_step_host_packed_async for the n layers of a model in one call: layer i
 * takes its inputs from host_in[i] and delivers to host_out[i] (host pointers to
 * pinned blocks laid out as segkv_host_pack_bytes says) without waiting.  The
 * launches go to `stream` in order; the copies travel on two streams of the
 * library's own, so that one layer's inputs arrive while the layer before it
 * computes, and `stream` ends behind the last copy out: waiting for `stream`
 * is waiting for every output.  (On a stream that is being captured everything
 * stays on `stream`.)  When the layers have the same shape and their blocks lie
 * back to back in host memory (host_in[i+1] = host_in[i] + block bytes, the same
 * for host_out: slices of one pinned array), several layers travel in one copy
 * each way through a staging area that the first layer's handle keeps; that area
 * is allocated at the first such call of a stack, which synchronises the device
 * once.  redo != 0 re-times a step: a handle whose newest
 * step is `step` drops it first (segkv_truncate_last) and takes it again.
 * No counterpart in the paper (an interface convenience: one call per decode
 * step instead of one per layer).  Errors: those of the single-layer call, at
 * the first layer that fails (earlier layers' work stays queued); EINVAL for
 * n <= 0 or NULL arrays.
 */
SEGKV_API int segkv_layers_step_host(const segkv_t* layers, int n, int step, const void* const* host_in,
                           void* const* host_out, int has_slopes, int redo, void* stream);


/* ---- test and benchmark aids ------------------------------------------- */

/* Forget all appended steps; keep_prompt == 0 also forgets the prompt. */
SEGKV_API int segkv_reset(segkv_t h, int keep_prompt);

/*
 * Drop the LAST appended step so that it can be appended again (used to time
 * a step repeatedly).  Only one step back is possible: the beam-index table
 * is updated incrementally and keeps one earlier generation.  ESTATE if no
 * step is appended or the previous call was also segkv_truncate_last.
 */
SEGKV_API int segkv_truncate_last(segkv_t h);

/* Copy the beam-index table to host_out [batch*beams][steps] (physical row in
 * [0,batch*beams) per beam slot and step).  Synchronises `stream`. */
SEGKV_API int segkv_get_ancestry(segkv_t h, int32_t* host_out, void* stream);

/* Per request, how many DISTINCT response rows its beams reference over all
 * appended steps (host_out [batch]); this is what the kernel reads.  Synchronises. */
SEGKV_API int segkv_get_unique_rows(segkv_t h, int32_t* host_out, void* stream);

/* Read and clear the device error word (SEGKV_DEV_* bits).  Synchronises the device. */
SEGKV_API int segkv_get_error(segkv_t h, int* device_flags);

/* Number of appended steps / current prompt length, or a negative error. */
SEGKV_API int segkv_steps(segkv_t h);
SEGKV_API int segkv_prompt_len(segkv_t h);

/*
 * Override the launch shape of the attention kernel: `splits` = CTAs that share
 * the keys of one (request, kv head) work group (at most 64), `stages` = depth
 * of the shared-memory ring, `combine` = how the splits are merged: 1 = partials
 * in a global workspace, merged by the last CTA to arrive; 2 = inside a
 * thread-block cluster through distributed shared memory (splits must be 2, 4
 * or 8).  0 = choose automatically from the shape (the default).  EINVAL if the
 * stages do not fit in shared memory; a forced cluster merge that the split
 * count does not allow is reported by the next segkv_decode_sdpa.
 * segkv_get_splits returns the split count the next segkv_decode_sdpa will use.
 */
SEGKV_API int segkv_set_tuning(segkv_t h, int splits, int stages, int combine);

/*
 * Pick the form of the decode attention kernel (a launch-shape knob: the paper
 * has no counterpart).  tile_keys = 64: tiles of 64 keys, four consumer warps,
 * two CTAs per SM (32 keys, two warps at head_dim 256): the form for launches
 * of several waves.  tile_keys = 32: tiles of 32 keys, two consumer warps, CTAs
 * of a quarter of an SM, so that the CTAs of two consecutive launches fit side
 * by side and the later one fetches its keys while the earlier one still
 * computes; only for head_dim <= 128 and beams*(heads/kv_heads) <= 8.
 * 0 = automatic (the default).  Errors: EINVAL (other values, or 32 for a shape
 * that has no such form).
 */
SEGKV_API int segkv_set_tile(segkv_t h, int tile_keys);

/*
 * Persistent form of segkv_decode_sdpa (a launch-shape knob: the paper has no
 * counterpart).  Instead of one CTA per (request, kv head, split), a grid of two
 * resident CTAs per SM walks those items round-robin, with the split count
 * chosen so that every CTA gets the same number of items: for launches between
 * one and a few waves of CTAs, whose last wave would otherwise leave SMs idle.
 * Results are those of segkv_decode_sdpa within the same tolerance (the keys
 * are grouped differently, so the low bits differ).  mode: -1 automatic (the
 * default), 0 never, 1 always.  Only for beams*(heads/kv_heads) <= 8; a split
 * count forced with segkv_set_tuning is used as the items per work group (at
 * most 8).  Errors: EINVAL (other values, or 1 for an unsupported shape).
 */
SEGKV_API int segkv_set_persistent(segkv_t h, int mode);
SEGKV_API int segkv_get_splits(segkv_t h);

/*
 * The same attention as segkv_decode_sdpa computed by the plain per-beam kernel
 * (each beam walks its own rows through the beam-index table, Section 3.3's
 * formulation taken literally; the prompt is re-read per beam).  Used for
 * shapes with more than 16 query columns per kv head, and as a cross-check.
 * Arguments and errors as segkv_decode_sdpa.
 */
SEGKV_API int segkv_decode_sdpa_rowwise(segkv_t h, const void* q, void* out, const float* alibi_slopes,
                                        void* stream);

/*
 * Programmatic dependent launch between the library's consecutive kernels on a
 * stream (on by default): a kernel may start while the previous one drains, and
 * the attention kernel requests its prompt tiles, which no decode-time call
 * modifies, before the previous kernel has finished; everything else is ordered
 * after it.  The first append after a prefill is always a fully serialised
 * launch.  enable == 0 turns it off (plain stream order).
 */
SEGKV_API int segkv_set_overlap(segkv_t h, int enable);

/*
 * segkv_append with the rotary position embedding applied to the new K rows on
 * their way into the response segment (Section 3.1 lists RoPE among the fused
 * kernels; here it rides on the copy the append does anyway).  Everything as
 * segkv_append, and:
 *   rope_cos, rope_sin: device float [rope_positions, head_dim/2]: cos and sin
 *     of the rotation angle of pair i at position m, row m of the table;
 *   style: SEGKV_ROPE_HALF pairs (x[i], x[i + head_dim/2]) (Llama, NeoX),
 *     SEGKV_ROPE_INTERLEAVED pairs (x[2i], x[2i+1]) (GPT-J); a pair (a, b)
 *     becomes (a cos - b sin, b cos + a sin), fp32 arithmetic, rounded once;
 *   the position of request b's token of this step is its prompt length + step.
 * V rows are stored as they come.  The query is NOT rotated by the library: q
 * handed to segkv_decode_sdpa must already carry its rotation.
 * Errors: those of segkv_append; EINVAL for NULL or misaligned tables or an
 * unknown style; ECAPACITY if a position would fall outside the tables.
 */
enum { SEGKV_ROPE_HALF = 1, SEGKV_ROPE_INTERLEAVED = 2 };
SEGKV_API int segkv_append_rope(segkv_t h, int step, const int32_t* beam_parent, const void* k_new,
                                const void* v_new, const float* rope_cos, const float* rope_sin,
                                int rope_positions, int style, void* stream);

/*
 * One set of beam-index tables for all layers of a model: the beam parents of
 * a step are the same for every layer, so only one handle (the leader) needs
 * to update the tables (Section 3.3's Indice table is kept by the beam search,
 * once).  After segkv_share_index(h, leader) the handle h
 *   - keeps its own prompt and response K/V, but reads the parent table, the
 *     beam-index table and the distinct-row lists of `leader`;
 *   - in segkv_append / segkv_append_rope stores its K/V rows only (the
 *     beam_parent argument is ignored); the leader must already have appended
 *     that step: ESTATE otherwise;
 *   - in segkv_decode_sdpa needs leader and h at the same step: ESTATE otherwise;
 *   - runs segkv_decode_step as those two launches.
 * Both handles must be at step 0 (ESTATE) and agree in batch, beams and
 * max_steps (EINVAL); a handle that follows cannot lead (EINVAL).
 * leader == NULL gives h its own tables back.  Truncating or resetting is the
 * caller's to do on every handle.  segkv_destroy of a handle that others still
 * follow returns ESTATE and destroys nothing: destroy the followers (or give
 * them their own tables back) first.
 */
SEGKV_API int segkv_share_index(segkv_t h, segkv_t leader);

/*
 * Memory layout of the prompt segment inside the handle (Section 4.1 / Fig. 6
 * of the paper compares prompt layouts for the decode kernel):
 *   SEGKV_PROMPT_HEAD_MAJOR  [batch, kv_heads, max_prompt, head_dim]  (default)
 *   SEGKV_PROMPT_TOKEN_MAJOR [batch, max_prompt, kv_heads, head_dim]  (the paper's [BS, Np, H, D])
 *   SEGKV_PROMPT_SEQ_FIRST   [max_prompt, batch, kv_heads, head_dim]  (sequence-first)
 * Every kernel reaches the prompt through a 4-D tensor map (or the strides) of
 * the chosen layout; results do not depend on it.  Only allowed while no prompt
 * is stored (before segkv_prefill_write, or after segkv_reset(h, 0)): ESTATE
 * otherwise; EINVAL for an unknown layout.  The inputs of segkv_prefill_write
 * stay token-major whatever the internal layout.
 */
enum { SEGKV_PROMPT_HEAD_MAJOR = 0, SEGKV_PROMPT_TOKEN_MAJOR = 1, SEGKV_PROMPT_SEQ_FIRST = 2 };
SEGKV_API int segkv_set_prompt_layout(segkv_t h, int layout);

/*
 * Override the CTA shape of the prefill attention kernel for head_dim 128
 * (the tcgen05 kernel): `row_groups` = groups of 128 query rows that one CTA
 * works on side by side (1 or 2; each group has its own softmax warps and
 * tensor-memory accumulators, all share the K/V tile ring).  0 = choose from
 * the grid size (the default).  EINVAL for any other value.  Other head sizes
 * ignore it.  A launch-shape knob: the paper has no counterpart.
 */
SEGKV_API int segkv_set_prefill_tuning(segkv_t h, int row_groups);

/*
 * Measurement aid (no counterpart in the paper): the bandwidth of a kernel that
 * only READS.  Streams `bytes` of device memory at dev_buf (16-byte aligned; use
 * a buffer several times the L2) `repeats` times with 16-byte loads, between two
 * CUDA events on `stream`, and returns GB/s in *gbs_out.  The decode attention
 * reads its keys and writes almost nothing, so this, not a copy's read+write
 * figure, is the ceiling its fraction of peak can be read against.  Allocates 256
 * bytes for the duration of the call and waits for the stream.
 * Errors: EINVAL, ECUDA.
 */
SEGKV_API int segkv_read_bandwidth(const void* dev_buf, size_t bytes, int repeats, float* gbs_out, void* stream);

/*
 * Test aid for the kernels' bounded waits (no counterpart in the paper).  Every
 * wait inside the attention kernels gives up after about two seconds, sets
 * SEGKV_DEV_WAIT_LIMIT in the device error word, lets copies in flight land,
 * releases what the kernel holds and returns without writing the output; the
 * call that launched it still returns SEGKV_OK and segkv_get_error() reports
 * the flag.  Nothing on a healthy device makes a wait run out, so a test asks
 * for it: the handle's NEXT attention launch (segkv_decode_sdpa,
 * segkv_decode_step's fused form, segkv_decode_sdpa_static or
 * segkv_prefill_sdpa) uses `wait_limit_ns` (0 = default) as the limit of its
 * waits and, if `skip_arrival` is non-zero, leaves out one plain mbarrier
 * arrival of one role (never a copy), so that the role waiting for it runs
 * into the limit.  The kernel returns by itself; later launches are normal.
 * Errors: EINVAL (NULL handle, negative limit).
 */
SEGKV_API int segkv_debug_inject(segkv_t h, long long wait_limit_ns, int skip_arrival);

/* Kernels launched by the handle since creation (each launch counted once). */
SEGKV_API long long segkv_launch_count(segkv_t h);

/*
 * K/V bytes one handle holds for the given shape: Eq. 3 of the paper for one
 * layer with the response capacity fixed at max_steps,
 *   batch * (max_prompt + beams*max_steps) * 2*kv_heads*head_dim*sizeof(dtype).
 * Pure host arithmetic; 0 on a bad argument.
 */
SEGKV_API size_t segkv_storage_bytes(int batch, int beams, int kv_heads, int head_dim, int max_prompt,
                           int max_steps, int dtype);

SEGKV_API const char* segkv_strerror(int code);
/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
SEGKV_API const char* segkv_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SEGKV_H */
