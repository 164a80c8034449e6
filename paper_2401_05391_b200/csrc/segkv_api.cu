// Host side of the segkv C-ABI: handle life cycle, argument checks, launches.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>

#include "segkv_internal.h"

using namespace segkv_impl;

namespace {

thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "%.120s: %.40s (%.80s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? SEGKV_ENOMEM : SEGKV_ECUDA;
}

#define SEGKV_CUDA(call)                                   \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

// ---------------------------------------------------------------------------
// Which of the library's launches came last on each stream.  A kernel launched with programmatic
// stream serialisation may begin before its predecessor P in the stream has finished, but not
// before P has passed its own grid-dependency wait, i.e. not before everything older than P is
// complete.  So data whose producing launch is strictly older than the latest library launch on
// the same stream may be read by the new kernel from its very first instruction.  (A launch of
// the caller's own in between only helps: it does not release its dependents early.)
// ---------------------------------------------------------------------------
struct StreamLog {
    cudaStream_t st;
    unsigned long long last;      // sequence number of the library's latest launch on st
    bool used;
};
std::mutex g_log_mu;
StreamLog g_log[32];
unsigned long long g_launch_seq = 0;

// Record a launch on `st`; returns its sequence number.
unsigned long long note_launch(cudaStream_t st) {
    std::lock_guard<std::mutex> lk(g_log_mu);
    const unsigned long long seq = ++g_launch_seq;
    int slot = -1, oldest = 0;
    for (int i = 0; i < 32; ++i) {
        if (g_log[i].used && g_log[i].st == st) { slot = i; break; }
        if (!g_log[i].used) { if (slot < 0) slot = i; }
        else if (g_log[i].last < g_log[oldest].last || !g_log[oldest].used) oldest = i;
    }
    if (slot < 0) slot = oldest;          // more than 32 streams: forget the one idle longest
    g_log[slot].st = st;
    g_log[slot].last = seq;
    g_log[slot].used = true;
    return seq;
}

// Is a launch `seq` on stream `st` strictly older than the library's latest launch there?
bool older_than_latest(cudaStream_t st, cudaStream_t seq_stream, unsigned long long seq) {
    if (seq == 0 || seq_stream != st) return false;
    std::lock_guard<std::mutex> lk(g_log_mu);
    for (int i = 0; i < 32; ++i)
        if (g_log[i].used && g_log[i].st == st) return seq < g_log[i].last;
    return false;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t elem_bytes(int dtype) { return (dtype == SEGKV_F16 || dtype == SEGKV_BF16) ? 2 : 0; }

bool dims_ok(int batch, int beams, int heads, int kv_heads, int head_dim, int max_prompt, int max_steps,
             int dtype) {
    if (batch <= 0 || beams <= 0 || heads <= 0 || kv_heads <= 0 || max_steps <= 0 || max_prompt < 0) return false;
    if (heads % kv_heads) return false;
    if (head_dim != 64 && head_dim != 128 && head_dim != 256) return false;
    if ((long long)beams * (heads / kv_heads) > kMaxCols) return false;
    if (elem_bytes(dtype) == 0) return false;
    return true;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// A 4-D tensor map in coordinates (d, head, token, request) over 16-bit elements: `heads` heads,
// `tokens` tokens (those past the extent read as zero), element strides of a head / token /
// request as given, box = 64 elements (128 bytes, one swizzle span) x box_tokens tokens of one
// (request, head), 128-byte swizzle.  `what` names the array in the error text.
int encode_map_4d(const segkv* h, const void* base, int heads, int tokens, long long stride_h, long long stride_p,
                  long long stride_b, int box_tokens, const char* what, CUtensorMap* out) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "cuTensorMapEncodeTiled entry point not available");
        return SEGKV_ECUDA;
    }
    const Dims& d = h->d;
    cuuint64_t dims[4] = {(cuuint64_t)d.head_dim, (cuuint64_t)heads, (cuuint64_t)tokens, (cuuint64_t)d.batch};
    cuuint64_t strides[3] = {(cuuint64_t)stride_h * 2, (cuuint64_t)stride_p * 2, (cuuint64_t)stride_b * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)box_tokens, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMapDataType dt = d.dtype == SEGKV_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    CUresult r = fn(out, dt, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "cuTensorMapEncodeTiled (%s) failed with CUresult %d", what, (int)r);
        return SEGKV_ECUDA;
    }
    return SEGKV_OK;
}

// One prompt array of the handle, [batch][prompt_len][kv_heads][D] logically, with the strides
// of the handle's prompt layout; a box is one tile of tokens.
int make_prompt_map(const segkv* h, void* base, int prompt_len, int box_tokens, CUtensorMap* out) {
    const PromptStrides ps = prompt_strides(h->d);
    return encode_map_4d(h, base, h->d.kv_heads, prompt_len, ps.h, ps.p, ps.b, box_tokens, "prompt segment", out);
}

// The handle's maps of its prompt segment: boxes of one regular tile (which the prefill kernel
// shares) and boxes of 32 tokens for the small-CTA form of the decode kernel.
int make_prompt_maps(segkv* h, int prompt_len) {
    const int box = tiled_tile_keys(h->d.head_dim, false);
    int rc = make_prompt_map(h, h->kp, prompt_len, box, &h->tm_kp);
    if (rc == SEGKV_OK) rc = make_prompt_map(h, h->vp, prompt_len, box, &h->tm_vp);
    if (rc == SEGKV_OK) rc = make_prompt_map(h, h->kp, prompt_len, 32, &h->tm_kp32);
    if (rc == SEGKV_OK) rc = make_prompt_map(h, h->vp, prompt_len, 32, &h->tm_vp32);
    return rc;
}

// The prefill query [batch][prompt_len][heads][D] (token-major): a box is 128 consecutive tokens.
int make_query_map(const segkv* h, const void* q, int prompt_len, CUtensorMap* out) {
    const long long D = h->d.head_dim, H = h->d.heads;
    return encode_map_4d(h, q, h->d.heads, prompt_len, D, D * H, D * H * prompt_len, 128, "prefill query", out);
}

// The caller's prefill K or V, token-major [batch][prompt_len][kv_heads][D], with the box of the
// prompt-segment maps.
int make_kv_source_map(const segkv* h, const void* base, int prompt_len, CUtensorMap* out) {
    const long long D = h->d.head_dim, Hkv = h->d.kv_heads;
    return encode_map_4d(h, base, h->d.kv_heads, prompt_len, D, D * Hkv, D * Hkv * prompt_len,
                         tiled_tile_keys(h->d.head_dim, false), "prefill K/V", out);
}

// Every kernel the library launches is counted on its handle and logged on its stream.
unsigned long long count_launch(segkv* h, cudaStream_t st) {
    h->launches++;
    return note_launch(st);
}

// The launch just made on `st` wrote the data `m` stands for.
void mark_written(segkv* h, WriteMark* m, cudaStream_t st) {
    m->seq = count_launch(h, st);
    m->stream = st;
}

// Is the data `m` stands for complete and visible to a kernel launched now on `st`, from that
// kernel's first instruction on?  Yes if its launch is strictly older than the library's latest
// launch on the same stream.  The answer depends on the order of the caller's calls alone, never on
// how far the GPU has got, so the same program takes the same path every time it runs.
bool settled(const WriteMark* m, cudaStream_t st) { return older_than_latest(st, m->stream, m->seq); }

void free_all(segkv* h) {
    void* ptrs[] = {h->kp, h->vp, h->kr, h->k_chunks_dev, h->parent, h->anc[0], h->anc[1], h->ulist, h->ucount, h->plens,
                    h->err_word, h->ws, h->tickets, h->st_q, h->st_out, h->st_k, h->st_v, h->st_parent, h->st_pack,
                    h->st_slopes, h->grp_in, h->grp_out};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    if (h->ev_in) cudaEventDestroy(h->ev_in);
    if (h->ev_k) cudaEventDestroy(h->ev_k);
    for (int c = 0; c < h->nchunks; ++c)
        if (h->k_chunks_host[c]) cudaFree(h->k_chunks_host[c]);
    free(h->k_chunks_host);
}

size_t slab_bytes_of(const Dims& d) { return (size_t)d.rows * d.kv_heads * d.head_dim * 2; }

// Device address of the K slab of response step `step` (its V slab is vdelta behind).
char* k_slab_of(const segkv* h, int step) {
    const Dims& d = h->d;
    if (d.chunk_steps == 0) return (char*)h->kr + (size_t)step * slab_bytes_of(d);
    const int c = step / d.chunk_steps;
    return (char*)h->k_chunks_host[c] + (size_t)(step - c * d.chunk_steps) * slab_bytes_of(d);
}

long long vdelta_of(const segkv* h) {
    const Dims& d = h->d;
    return (long long)((size_t)(d.chunk_steps ? d.chunk_steps : d.max_steps) * slab_bytes_of(d));
}

// Growing capacity (Section 3.2): make sure the chunk that holds `step` exists.  A new chunk is
// one allocation {K part, V part}; its address is appended to the device table on the stream.
int ensure_chunk(segkv* h, int step, cudaStream_t st) {
    const Dims& d = h->d;
    if (d.chunk_steps == 0) return SEGKV_OK;
    const int need = step / d.chunk_steps + 1;
    while (h->nchunks < need) {
        void* p = nullptr;
        SEGKV_CUDA(cudaMalloc(&p, 2 * (size_t)d.chunk_steps * slab_bytes_of(d)));
        h->k_chunks_host[h->nchunks] = p;
        SEGKV_CUDA(cudaMemcpyAsync(h->k_chunks_dev + h->nchunks, h->k_chunks_host + h->nchunks, sizeof(void*),
                                   cudaMemcpyHostToDevice, st));
        h->nchunks++;
    }
    return SEGKV_OK;
}

template <typename T>
cudaError_t dmalloc(T** p, size_t bytes) {
    return cudaMalloc((void**)p, bytes ? bytes : 16);
}

int alloc_workspace(segkv* h, int splits) {
    const Dims& d = h->d;
    size_t cols = (size_t)d.beams * d.group;
    size_t bytes = (size_t)d.batch * d.kv_heads * splits * cols * (d.head_dim + 2) * sizeof(float);
    if (h->ws) {
        cudaFree(h->ws);
        h->ws = nullptr;
    }
    SEGKV_CUDA(dmalloc(&h->ws, bytes));
    h->ws_bytes = bytes;
    h->ws_splits = splits;
    return SEGKV_OK;
}

// Launch shape of the tiled kernel.
struct Tiling {
    int splits, stages;
    bool one_wave;    // all CTAs of the launch fit on the GPU at once and have only a few tiles each
    bool cluster;     // the splits of a work group merge inside a thread-block cluster
    bool small;       // 32-key tiles, quarter-SM CTAs
    int tail_groups, tail_splits;   // the work groups of a ragged last wave, cut finer so that they cover all SMs
};

// CTAs of the chosen form that one SM holds at once.
int ctas_per_sm(bool small) { return small ? 4 : 2; }

// Most splits the automatic choice makes for this handle (what the split workspace is sized for).
int max_auto_splits(const segkv* h) {
    const long long slabs = (long long)h->d.batch * h->d.kv_heads;
    long long most = (long long)h->sm_count * 4 / slabs;
    if (most < 1) most = 1;
    return (int)(most > kMaxSplits ? kMaxSplits : most);
}

// Stages: as many as keep the form's CTAs per SM resident.  Splits: none when the work groups
// alone fill the GPU twice over, else enough to give every CTA slot of one wave a share (never
// less than one tile each).
Tiling choose_tiling(const segkv* h, bool fused_step) {
    const Dims& d = h->d;
    Tiling t;
    // A launch of eight splits that fills about half of the GPU's quarter-SM slots runs in the
    // small-CTA form, its splits merged inside a thread-block cluster: the next launch's CTAs then
    // fit beside this one's and fetch their keys while these still compute (measured at the
    // Llama2-7B shape: fused step 7.6 us per layer against 9.6 us in the regular form, the attention
    // call on its own 6.5 against 7.4 us; at the Llama2-13B shape, 320 CTAs, where the next launch
    // only fits in part: 9.1 against 10.6 us).  Larger launches keep the regular form.  (A chain of
    // launches of 320 CTAs in clusters of FOUR, eight prompt tiles per CTA, once ended in a launch
    // failure on two of three runs; that was before a stage's release waited for both consumer warps,
    // the shape has not been run since and this rule never makes it.)
    if (h->tile_forced == 0 && h->splits_forced <= 0 && h->stages_forced <= 0 && h->combine_forced != 1 &&
        h->overlap && tiled_small_ok(d) && (h->prompt_len >= 8 * 32 || h->steps >= 16)) {     // work for eight CTAs
        const long long slabs = (long long)d.batch * d.kv_heads;
        // (up to six 32-key prompt tiles per CTA: with more, the CTAs stream and the regular form's larger
        // tiles and deeper ring win: prompt 4096 at the Llama2-13B shape 19.0 against 24.8 us)
        if (slabs * 8 <= 2LL * h->sm_count + h->sm_count / 4 && tiled_cluster_ok(d, 8) && h->prompt_len <= 6 * 8 * 32) {
            t.small = true;
            t.cluster = true;
            t.one_wave = true;
            t.tail_groups = t.tail_splits = 0;
            t.splits = 8;
            t.stages = 2;
            const size_t budget = (h->smem_optin + 1024) / ctas_per_sm(true) - 1024;
            while (t.stages < 8 && tiled_smem_bytes(d, t.stages + 1, true) <= budget) ++t.stages;
            return t;
        }
    }
    t.small = h->tile_forced == 32 && tiled_small_ok(d);
    {
        // Between half a wave and two waves of the regular form's CTA slots, one CTA per work group
        // leaves slots idle or a ragged second wave (measured at the Llama2-13B shape: 0.67-0.69 of the
        // copy bandwidth at batch 4 and 8).  The small-CTA form has twice the slots: as many splits as
        // still make one wave of them (0.76 and 0.83 there).
        const long long slabs = (long long)d.batch * d.kv_heads;
        const long long slots_small = (long long)h->sm_count * ctas_per_sm(true);
        const long long slots_regular = (long long)h->sm_count * ctas_per_sm(false);
        // (work groups that fill two thirds or more of ONE wave of the regular form are best left alone, one
        // regular CTA each: 0.76 / 0.82 / 0.86 at batch 5 / 6 / 7 against 0.71 / 0.76 / 0.80 in the small form)
        const bool one_regular_wave = 3 * slabs >= 2 * slots_regular && slabs <= slots_regular;
        // Beyond one wave of them the small form stays ahead as well (Llama2-13B shape, batch 16 to 64: 0.94-1.05
        // of the copy bandwidth against 0.88-1.01; OPT-30B shape 606 against 611 us): more, smaller CTAs leave
        // a shorter ragged end.
        if (h->tile_forced == 0 && h->splits_forced <= 0 && tiled_small_ok(d) && slabs > h->sm_count && !one_regular_wave)
            t.small = true;
        (void)slots_small;
    }
    const int tile = tiled_tile_keys(d.head_dim, t.small);
    const int P = h->prompt_len > 0 ? h->prompt_len : 0;
    const long long ntp = (P + tile - 1) / tile;
    const long long ntr = (h->steps + 2 * d.beams + tile - 1) / tile;      // estimate, rows are mostly shared
    const long long slabs = (long long)d.batch * d.kv_heads;
    const long long slots = (long long)h->sm_count * ctas_per_sm(t.small);
    int sp = h->splits_forced;
    if (sp <= 0) {
        sp = 1;
        if (slabs < 2 * slots) {
            long long want = slots / slabs;
            if (want > ntp + ntr) want = ntp + ntr;
            if (want < 1) want = 1;
            // the fewest splits that reach the same number of prompt tiles per CTA
            const long long per = ntp > 0 ? (ntp + want - 1) / want : 1;
            long long s = ntp > 0 ? (ntp + per - 1) / per : want;
            if (s > kMaxSplits) s = kMaxSplits;
            sp = (int)s;
        }
    }
    if (sp > kMaxSplits) sp = kMaxSplits;
    int st = h->stages_forced;
    if (st <= 0) {
        // as deep a ring as still lets the form's CTAs share an SM ...
        st = 2;
        const size_t budget = (h->smem_optin + 1024) / ctas_per_sm(t.small) - 1024 - (t.small ? 0 : 2048);
        while (st < 8 && tiled_smem_bytes(d, st + 1, t.small) <= budget) ++st;
        // ... or, when the whole launch is one wave, deep enough to hold a CTA's whole share
        const long long per_cta = (ntp + sp - 1) / sp + (ntr + sp - 1) / sp;
        if (!t.small && slabs * sp <= h->sm_count && per_cta > st) {
            while (st < per_cta && st < 8 && tiled_smem_bytes(d, st + 1, t.small) <= h->smem_optin) ++st;
        }
    }
    while (st > 1 && tiled_smem_bytes(d, st, t.small) > h->smem_optin) --st;
    t.splits = sp;
    t.stages = st;
    // "one wave" in the sense that matters: every CTA resident at once AND a share of a few tiles each,
    // i.e. a launch whose time is its chain of latencies, not the bytes it moves
    t.one_wave = slabs * sp <= slots && (ntp + sp - 1) / sp <= 2 * st;
    // The workspace merge is the default: launches that merge inside a cluster were measured
    // not to start early under programmatic dependent launch, which costs more than the
    // cluster merge saves.  With overlap off the cluster merge is the faster one.
    const bool want_cluster = h->combine_forced == 2 || (h->combine_forced == 0 && !h->overlap);
    t.cluster = sp > 1 && want_cluster && tiled_cluster_ok(d, sp);
    // More work groups than CTA slots, one CTA each, and a last wave that fills at most half of the slots:
    // that wave alone would take as long as a full one (Llama2-13B shape at batch 16: 640 CTAs on 296 slots,
    // 0.78 of the copy bandwidth).  Its work groups are cut into as many splits as spread them over all slots;
    // they are the last CTAs of the grid, so they start when the full waves drain.
    t.tail_groups = t.tail_splits = 0;
    if (!fused_step && sp == 1 && h->splits_forced <= 0 && !t.cluster && slabs > slots) {
        const long long r = slabs % slots;
        if (r > 0 && 2 * r <= slots) {
            long long s = slots / r;
            if (s > 8) s = 8;
            if (s > ntp / 2) s = ntp / 2;          // at least two prompt tiles per CTA
            if (s >= 2) {
                t.tail_groups = (int)r;
                t.tail_splits = (int)s;
            }
        }
    }
    return t;
}

// Items per work group for the persistent form: the split count (at most 4, at least two prompt tiles
// per item) whose items deal most evenly over the resident grid; ties go to fewer splits.
int stream_splits(const segkv* h) {
    if (h->splits_forced > 0) return h->splits_forced > 8 ? 8 : h->splits_forced;
    const Dims& d = h->d;
    const long long slabs = (long long)d.batch * d.kv_heads;
    const long long grid = (long long)h->sm_count * stream_ctas_per_sm();
    const int tile = tiled_tile_keys(d.head_dim, false);
    const long long ntp = ((h->prompt_len > 0 ? h->prompt_len : 0) + tile - 1) / tile;
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= 4; ++s) {
        if (s > 1 && ntp / s < 2) break;
        const long long items = slabs * s;
        const long long rounds = (items + grid - 1) / grid;
        const double eff = (double)items / (double)(rounds * grid) - 0.02 * (s - 1);
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best = s;
        }
    }
    return best;
}

// Does the separate attention call run in the persistent form?
bool use_stream(const segkv* h) {
    if (h->persist_mode == 0 || !stream_supported(h->d) || h->tile_forced != 0 || h->combine_forced == 2) return false;
    if (h->persist_mode == 1) return true;
    return false;
}

// The attention kernel's separate form walks per-request lists of distinct rows that the append
// kernel makes; fused steps skip them, so they are re-derived from the table when needed.
// The handle that owns the beam-index tables h works with.
segkv* index_of(segkv* h) { return h->leader ? h->leader : h; }
const segkv* index_of(const segkv* h) { return h->leader ? h->leader : h; }

int ensure_lists(segkv* h, cudaStream_t st) {
    segkv* x = index_of(h);
    if (x->lists_valid || h->steps == 0) return SEGKV_OK;
    SEGKV_CUDA(launch_rebuild_lists(x->d, h->steps, x->anc[(h->steps - 1) & 1], x->ulist, x->ucount, st));
    mark_written(h, &x->lists_mark, st);
    x->lists_valid = true;
    return SEGKV_OK;
}

// May the next attention launch on `st` read the handle's response rows (and, for the separate
// form, the distinct-row lists) before its grid-dependency wait?  Only if the launches that wrote
// them are strictly older than the library's latest launch on the same stream.
bool rows_settled(const segkv* h, cudaStream_t st, bool lists_too) {
    if (!h->overlap || h->steps == 0) return false;
    if (!settled(&h->rows_mark, st)) return false;
    if (!lists_too) return true;
    return settled(&index_of(h)->lists_mark, st);
}

SdpaArgs sdpa_args(const segkv* h, const void* q, void* out, const float* slopes, int splits) {
    SdpaArgs a;
    a.q = q;
    a.out = out;
    a.slopes = slopes;
    a.kp = h->kp;
    a.vp = h->vp;
    a.kr = h->kr;
    a.vr = h->vr;
    a.k_chunks = (const void* const*)h->k_chunks_dev;
    a.vdelta = vdelta_of(h);
    const segkv* x = index_of(h);
    a.anc = x->anc[h->steps > 0 ? ((h->steps - 1) & 1) : 0];
    a.ulist = x->ulist;
    a.ucount = x->ucount;
    a.plens = h->ragged ? h->plens : nullptr;
    a.ws = h->ws;
    a.tickets = h->tickets;
    a.err_word = h->err_word;
    a.prompt_len = h->prompt_len > 0 ? h->prompt_len : 0;
    a.steps = h->steps;
    a.splits = splits;
    a.tail_groups = a.tail_splits = 0;
    a.cluster = false;
    a.small = false;
    a.one_wave = false;
    a.pdl = false;
    a.prompt_immutable = h->steps > 0;     // the first append after a prefill is a fully serialised launch
    a.rows_immutable = false;
    a.fused = false;
    a.wait_ns = h->dbg_wait_ns;
    a.dbg_skip = h->dbg_skip;
    a.parent = nullptr;
    a.k_new = a.v_new = nullptr;
    a.kr_new_slab = a.vr_new_slab = nullptr;
    a.anc_dst = nullptr;
    a.parent_row = nullptr;
    return a;
}

}  // namespace

extern "C" {

size_t segkv_storage_bytes(int batch, int beams, int kv_heads, int head_dim, int max_prompt, int max_steps,
                           int dtype) {
    if (batch <= 0 || beams <= 0 || kv_heads <= 0 || head_dim <= 0 || max_prompt < 0 || max_steps < 0) return 0;
    size_t eb = elem_bytes(dtype);
    if (!eb) return 0;
    size_t token = 2 * (size_t)kv_heads * head_dim * eb;
    return (size_t)batch * ((size_t)max_prompt + (size_t)beams * max_steps) * token;
}

long long segkv_allocated_kv_bytes(segkv_t h) {
    if (!h) return SEGKV_EINVAL;
    const Dims& d = h->d;
    const size_t token = 2 * (size_t)d.kv_heads * d.head_dim * 2;
    const size_t steps_held = d.chunk_steps ? (size_t)h->nchunks * d.chunk_steps : (size_t)d.max_steps;
    return (long long)((size_t)d.batch * ((size_t)d.max_prompt + (size_t)d.beams * steps_held) * token);
}

const char* segkv_strerror(int code) {
    switch (code) {
        case SEGKV_OK: return "ok";
        case SEGKV_EINVAL: return "invalid argument";
        case SEGKV_ESTATE: return "call out of order for the handle's state";
        case SEGKV_ECAPACITY: return "beyond the capacity given at segkv_create";
        case SEGKV_ENOMEM: return "out of memory";
        case SEGKV_ECUDA: return "CUDA error (see segkv_last_cuda_error)";
        case SEGKV_EDEVICE: return "a kernel reported an error (see segkv_get_error)";
        default: return "unknown segkv error code";
    }
}

const char* segkv_last_cuda_error(void) { return g_cuda_err; }

int segkv_create(segkv_t* out, int batch, int beams, int heads, int kv_heads, int head_dim, int max_prompt,
                 int max_steps, int dtype) {
    return segkv_create_growing(out, batch, beams, heads, kv_heads, head_dim, max_prompt, max_steps, 0, dtype);
}

int segkv_create_growing(segkv_t* out, int batch, int beams, int heads, int kv_heads, int head_dim, int max_prompt,
                         int max_steps, int chunk_steps, int dtype) {
    if (!out) return SEGKV_EINVAL;
    if (!dims_ok(batch, beams, heads, kv_heads, head_dim, max_prompt, max_steps, dtype)) return SEGKV_EINVAL;
    if (chunk_steps < 0) return SEGKV_EINVAL;
    if (chunk_steps >= max_steps) chunk_steps = 0;      // one chunk would hold everything: fixed capacity
    segkv* h = new (std::nothrow) segkv();
    if (!h) return SEGKV_ENOMEM;
    memset(h, 0, sizeof *h);
    Dims& d = h->d;
    d.batch = batch; d.beams = beams; d.heads = heads; d.kv_heads = kv_heads; d.head_dim = head_dim;
    d.group = heads / kv_heads; d.max_prompt = max_prompt; d.max_steps = max_steps;
    d.rows = batch * beams; d.dtype = dtype; d.chunk_steps = chunk_steps;
    h->prompt_len = -1;
    h->overlap = true;
    h->persist_mode = -1;
    h->prefill_groups = 0;
    h->ragged = false;
    h->leader = nullptr;
    h->followers = 0;
    d.prompt_layout = SEGKV_PROMPT_HEAD_MAJOR;

    int rc = SEGKV_OK;
    auto fail = [&](int code) { free_all(h); delete h; return code; };
#define SEGKV_TRY(call)                                     \
    do {                                                    \
        cudaError_t e__ = (call);                           \
        if (e__ != cudaSuccess) return fail(cuda_fail(e__, #call)); \
    } while (0)
    SEGKV_TRY(cudaGetDevice(&h->device));
    SEGKV_TRY(cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device));
    int optin = 0;
    SEGKV_TRY(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device));
    h->smem_optin = (size_t)optin;

    const size_t eb = 2;
    const size_t prompt_bytes = (size_t)batch * kv_heads * max_prompt * head_dim * eb;
    const size_t resp_bytes = (size_t)max_steps * d.rows * kv_heads * head_dim * eb;
    SEGKV_TRY(dmalloc(&h->kp, prompt_bytes));
    SEGKV_TRY(dmalloc(&h->vp, prompt_bytes));
    if (chunk_steps == 0) {
        SEGKV_TRY(dmalloc(&h->kr, 2 * resp_bytes));                      // K, then V, in one allocation
        h->vr = (char*)h->kr + resp_bytes;
    } else {
        h->nchunks_max = (max_steps + chunk_steps - 1) / chunk_steps;
        h->k_chunks_host = (void**)calloc((size_t)h->nchunks_max, sizeof(void*));
        if (!h->k_chunks_host) return fail(SEGKV_ENOMEM);
        SEGKV_TRY(dmalloc(&h->k_chunks_dev, (size_t)h->nchunks_max * sizeof(void*)));
    }
    SEGKV_TRY(dmalloc(&h->parent, (size_t)max_steps * d.rows * sizeof(int32_t)));
    SEGKV_TRY(dmalloc(&h->anc[0], (size_t)max_steps * d.rows * sizeof(int32_t)));
    SEGKV_TRY(dmalloc(&h->anc[1], (size_t)max_steps * d.rows * sizeof(int32_t)));
    SEGKV_TRY(dmalloc(&h->ulist, (size_t)max_steps * d.rows * sizeof(URow)));
    SEGKV_TRY(dmalloc(&h->ucount, (size_t)batch * sizeof(int32_t)));
    SEGKV_TRY(cudaMemset(h->ucount, 0, (size_t)batch * sizeof(int32_t)));
    SEGKV_TRY(dmalloc(&h->plens, (size_t)batch * sizeof(int32_t)));
    SEGKV_TRY(dmalloc(&h->err_word, sizeof(int)));
    SEGKV_TRY(dmalloc(&h->tickets, (size_t)batch * kv_heads * sizeof(int)));
    SEGKV_TRY(cudaMemset(h->err_word, 0, sizeof(int)));
    SEGKV_TRY(cudaMemset(h->tickets, 0, (size_t)batch * kv_heads * sizeof(int)));
    const size_t qbytes = (size_t)d.rows * heads * head_dim * eb;
    const size_t kvbytes = (size_t)d.rows * kv_heads * head_dim * eb;
    SEGKV_TRY(dmalloc(&h->st_q, qbytes));
    SEGKV_TRY(dmalloc(&h->st_out, qbytes));
    SEGKV_TRY(dmalloc(&h->st_k, kvbytes));
    SEGKV_TRY(dmalloc(&h->st_v, kvbytes));
    SEGKV_TRY(dmalloc(&h->st_parent, (size_t)d.rows * sizeof(int32_t)));
    SEGKV_TRY(dmalloc(&h->st_slopes, (size_t)heads * sizeof(float)));
    SEGKV_TRY(dmalloc(&h->st_pack, segkv_host_pack_bytes(h, nullptr)));
#undef SEGKV_TRY
    // The split workspace for the largest split count the automatic choice can make (one wave of
    // CTA slots shared among the work groups), so that the decode loop never allocates.
    if (cudaEventCreateWithFlags(&h->ev_in, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_k, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        return fail(SEGKV_ECUDA);
    }
    rc = alloc_workspace(h, max_auto_splits(h));
    if (rc != SEGKV_OK) return fail(rc);
    *out = h;
    return SEGKV_OK;
}

int segkv_destroy(segkv_t h) {
    if (!h) return SEGKV_OK;
    if (h->followers > 0) return SEGKV_ESTATE;        // other handles still read this one's tables
    if (h->leader) h->leader->followers--;
    cudaDeviceSynchronize();
    free_all(h);
    delete h;
    return SEGKV_OK;
}

static int prefill_write_impl(segkv_t h, const void* k, const void* v, int prompt_len, const int32_t* plens_dev,
                              void* stream);

int segkv_prefill_write(segkv_t h, const void* k, const void* v, int prompt_len, void* stream) {
    if (!h) return SEGKV_EINVAL;
    int rc = prefill_write_impl(h, k, v, prompt_len, nullptr, stream);
    if (rc == SEGKV_OK) h->ragged = false;
    return rc;
}

int segkv_prefill_write_ragged(segkv_t h, const void* k, const void* v, int padded_len, const int32_t* prompt_lens,
                               void* stream) {
    if (!h || !prompt_lens || padded_len <= 0) return SEGKV_EINVAL;
    if (padded_len > h->d.max_prompt) return SEGKV_ECAPACITY;
    for (int b = 0; b < h->d.batch; ++b)
        if (prompt_lens[b] < 1 || prompt_lens[b] > padded_len) return SEGKV_EINVAL;
    // the lengths travel on the caller's stream, ahead of the kernel that reads them; the source
    // is pageable host memory, so the copy has been staged by the time the call returns
    SEGKV_CUDA(cudaMemcpyAsync(h->plens, prompt_lens, (size_t)h->d.batch * sizeof(int32_t), cudaMemcpyHostToDevice,
                               (cudaStream_t)stream));
    int rc = prefill_write_impl(h, k, v, padded_len, h->plens, stream);
    if (rc == SEGKV_OK) h->ragged = true;
    return rc;
}

static int prefill_write_impl(segkv_t h, const void* k, const void* v, int prompt_len, const int32_t* plens_dev,
                              void* stream) {
    if (!h || prompt_len < 0) return SEGKV_EINVAL;
    if (prompt_len > h->d.max_prompt) return SEGKV_ECAPACITY;
    if (prompt_len > 0 && (!k || !v || !aligned16(k) || !aligned16(v))) return SEGKV_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    h->tm_valid = false;
    if (prompt_len > 0) {
        SEGKV_CUDA(launch_prefill_transpose(h->d, k, v, h->kp, h->vp, plens_dev, prompt_len, h->sm_count, st));
        count_launch(h, st);
        int rc = make_prompt_maps(h, prompt_len);
        if (rc != SEGKV_OK) return rc;
        h->tm_valid = true;
    }
    h->prompt_len = prompt_len;
    h->steps = 0;
    h->truncated = false;
    return SEGKV_OK;
}

int segkv_prefill_sdpa(segkv_t h, const void* q, void* out, const float* alibi_slopes, void* stream) {
    if (!h || !q || !out || !aligned16(q) || !aligned16(out)) return SEGKV_EINVAL;
    if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SEGKV_EINVAL;
    if (h->prompt_len <= 0 || !h->tm_valid) return SEGKV_ESTATE;
    if (!prefill_tc5_supported(h->d)) return SEGKV_EINVAL;
    PrefillArgs a;
    a.q = q; a.out = out; a.slopes = alibi_slopes; a.err_word = h->err_word;
    a.prompt_len = h->prompt_len; a.tm_k = &h->tm_kp; a.tm_v = &h->tm_vp;
    a.row_groups = h->prefill_groups;
    a.wait_ns = h->dbg_wait_ns;
    a.dbg_skip = h->dbg_skip;
    h->dbg_wait_ns = 0;
    h->dbg_skip = false;
    a.plens = h->ragged ? h->plens : nullptr;
    a.tm_k_src = a.tm_v_src = nullptr;
    CUtensorMap tm_q;
    a.tm_q = nullptr;
    if (prefill_tc5_supported(h->d)) {
        int rc = make_query_map(h, q, h->prompt_len, &tm_q);
        if (rc != SEGKV_OK) return rc;
        a.tm_q = &tm_q;
    }
    SEGKV_CUDA(launch_prefill_tc5(h->d, a, (cudaStream_t)stream));
    count_launch(h, (cudaStream_t)stream);
    return SEGKV_OK;
}

int segkv_prefill(segkv_t h, const void* k, const void* v, const void* q, void* out, int prompt_len,
                  const float* alibi_slopes, void* stream) {
    if (!h) return SEGKV_EINVAL;
    if (prompt_len <= 0 || !prefill_tc5_supported(h->d)) {
        int rc = segkv_prefill_write(h, k, v, prompt_len, stream);
        if (rc != SEGKV_OK) return rc;
        return segkv_prefill_sdpa(h, q, out, alibi_slopes, stream);
    }
    // One launch: the attention kernel reads K/V from the caller's arrays and stores every tile
    // into the prompt segment on the way (each tile by exactly one CTA), instead of a copy kernel
    // first and the attention over the copy after it.
    if (!k || !v || !q || !out || !aligned16(k) || !aligned16(v) || !aligned16(q) || !aligned16(out)) return SEGKV_EINVAL;
    if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SEGKV_EINVAL;
    if (prompt_len > h->d.max_prompt) return SEGKV_ECAPACITY;
    h->tm_valid = false;
    int rc = make_prompt_maps(h, prompt_len);
    CUtensorMap tm_q, tm_ks, tm_vs;
    if (rc == SEGKV_OK) rc = make_kv_source_map(h, k, prompt_len, &tm_ks);
    if (rc == SEGKV_OK) rc = make_kv_source_map(h, v, prompt_len, &tm_vs);
    if (rc == SEGKV_OK) rc = make_query_map(h, q, prompt_len, &tm_q);
    if (rc != SEGKV_OK) return rc;
    PrefillArgs a;
    a.q = q; a.out = out; a.slopes = alibi_slopes; a.err_word = h->err_word;
    a.prompt_len = prompt_len; a.tm_k = &h->tm_kp; a.tm_v = &h->tm_vp;
    a.row_groups = h->prefill_groups;
    a.wait_ns = 0;
    a.dbg_skip = false;
    a.plens = nullptr;
    a.tm_k_src = &tm_ks; a.tm_v_src = &tm_vs; a.tm_q = &tm_q;
    h->prompt_len = -1;                                       // nothing valid is stored if the launch fails
    SEGKV_CUDA(launch_prefill_tc5(h->d, a, (cudaStream_t)stream));
    count_launch(h, (cudaStream_t)stream);
    h->tm_valid = true;
    h->prompt_len = prompt_len;
    h->steps = 0;
    h->truncated = false;
    h->ragged = false;
    return SEGKV_OK;
}

static int append_impl(segkv_t h, int step, const int32_t* beam_parent, const void* k_new, const void* v_new,
                       const RopeArgs* rope, void* stream);

int segkv_append(segkv_t h, int step, const int32_t* beam_parent, const void* k_new, const void* v_new,
                 void* stream) {
    return append_impl(h, step, beam_parent, k_new, v_new, nullptr, stream);
}

int segkv_append_rope(segkv_t h, int step, const int32_t* beam_parent, const void* k_new, const void* v_new,
                      const float* rope_cos, const float* rope_sin, int rope_positions, int style, void* stream) {
    if (!h || !rope_cos || !rope_sin || rope_positions <= 0) return SEGKV_EINVAL;
    if (style != SEGKV_ROPE_HALF && style != SEGKV_ROPE_INTERLEAVED) return SEGKV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(rope_cos) & 3u) || (reinterpret_cast<uintptr_t>(rope_sin) & 3u)) return SEGKV_EINVAL;
    if (h->prompt_len < 0) return SEGKV_ESTATE;
    if (step >= 0 && h->prompt_len + step >= rope_positions) return SEGKV_ECAPACITY;   // the longest request's position
    RopeArgs r;
    r.cos = rope_cos; r.sin = rope_sin;
    r.plens = h->ragged ? h->plens : nullptr;
    r.prompt_len = h->prompt_len;
    r.style = style;
    r.head_dim = h->d.head_dim; r.kv_heads = h->d.kv_heads; r.bf16 = h->d.dtype == SEGKV_BF16;
    return append_impl(h, step, beam_parent, k_new, v_new, &r, stream);
}

static int append_impl(segkv_t h, int step, const int32_t* beam_parent, const void* k_new, const void* v_new,
                       const RopeArgs* rope, void* stream) {
    if (!h || step < 0 || !k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return SEGKV_EINVAL;
    if (step > 0 && (!beam_parent || (reinterpret_cast<uintptr_t>(beam_parent) & 3u))) return SEGKV_EINVAL;
    if (h->prompt_len < 0) return SEGKV_ESTATE;
    if (step != h->steps) return SEGKV_ESTATE;
    if (step >= h->d.max_steps) return SEGKV_ECAPACITY;
    {
        int rc = ensure_chunk(h, step, (cudaStream_t)stream);
        if (rc != SEGKV_OK) return rc;
    }
    if (h->leader) {
        // the tables of this step have been made by the leader's call: only the K/V rows are stored
        if (h->leader->steps != step + 1 || h->leader->truncated) return SEGKV_ESTATE;
        SEGKV_CUDA(launch_append(h->d, step, nullptr, k_new, v_new, k_slab_of(h, step),
                                 k_slab_of(h, step) + vdelta_of(h), nullptr, nullptr, nullptr, nullptr, nullptr,
                                 h->err_word, h->sm_count, h->overlap && step > 0, (cudaStream_t)stream, rope, false));
        mark_written(h, &h->rows_mark, (cudaStream_t)stream);
        h->steps = step + 1;
        h->truncated = false;
        return SEGKV_OK;
    }
    SEGKV_CUDA(launch_append(h->d, step, beam_parent, k_new, v_new, k_slab_of(h, step),
                             k_slab_of(h, step) + vdelta_of(h), h->parent,
                             h->anc[(step + 1) & 1], h->anc[step & 1], h->ulist, h->ucount, h->err_word,
                             h->sm_count, h->overlap && step > 0, (cudaStream_t)stream, rope));
    mark_written(h, &h->rows_mark, (cudaStream_t)stream);
    h->lists_mark = h->rows_mark;                  // the same launch made the lists
    h->steps = step + 1;
    h->truncated = false;
    h->lists_valid = true;
    return SEGKV_OK;
}

int segkv_decode_sdpa(segkv_t h, const void* q, void* out, const float* alibi_slopes, void* stream) {
    if (!h || !q || !out || !aligned16(q) || !aligned16(out)) return SEGKV_EINVAL;
    if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SEGKV_EINVAL;
    if (h->prompt_len < 0) return SEGKV_ESTATE;
    if (h->prompt_len + h->steps <= 0) return SEGKV_ESTATE;
    if (h->leader && h->leader->steps != h->steps) return SEGKV_ESTATE;   // the shared tables describe another step
    if (!tiled_supported(h->d)) {
        SdpaArgs a = sdpa_args(h, q, out, alibi_slopes, 1);
        SEGKV_CUDA(launch_sdpa_rowwise(h->d, a, (cudaStream_t)stream));
        count_launch(h, (cudaStream_t)stream);
        return SEGKV_OK;
    }
    {
        int rc = ensure_lists(h, (cudaStream_t)stream);
        if (rc != SEGKV_OK) return rc;
    }
    if (use_stream(h)) {
        const int sp = stream_splits(h);
        if (sp > h->ws_splits) {
            SEGKV_CUDA(cudaDeviceSynchronize());
            int rc = alloc_workspace(h, sp);
            if (rc != SEGKV_OK) return rc;
        }
        SdpaArgs a = sdpa_args(h, q, out, alibi_slopes, sp);
        a.pdl = h->overlap;
        h->dbg_wait_ns = 0;
        h->dbg_skip = false;
        SEGKV_CUDA(launch_sdpa_stream(h->d, a, h->tm_kp, h->tm_vp, h->sm_count, (cudaStream_t)stream));
        count_launch(h, (cudaStream_t)stream);
        return SEGKV_OK;
    }
    const Tiling tl = choose_tiling(h, false);
    const int splits = tl.splits;
    if (h->combine_forced == 2 && splits > 1 && !tl.cluster) return SEGKV_EINVAL;
    if (!tl.cluster && splits > h->ws_splits) {
        // growing the workspace must not race with work still using the old one
        SEGKV_CUDA(cudaDeviceSynchronize());
        int rc = alloc_workspace(h, splits);
        if (rc != SEGKV_OK) return rc;
    }
    SdpaArgs a = sdpa_args(h, q, out, alibi_slopes, splits);
    a.cluster = tl.cluster;
    a.small = tl.small;
    a.one_wave = tl.one_wave;
    a.tail_groups = tl.tail_groups;
    a.tail_splits = tl.tail_splits;
    a.pdl = h->overlap;
    a.rows_immutable = rows_settled(h, (cudaStream_t)stream, true);
    h->dbg_wait_ns = 0;                  // an injected fault applies to one launch
    h->dbg_skip = false;
    SEGKV_CUDA(launch_sdpa_tiled(h->d, a, tl.small ? h->tm_kp32 : h->tm_kp, tl.small ? h->tm_vp32 : h->tm_vp, tl.stages,
                                 (cudaStream_t)stream));
    count_launch(h, (cudaStream_t)stream);
    return SEGKV_OK;
}

int segkv_decode_sdpa_static(segkv_t h, const void* q, void* out, const float* alibi_slopes, void* stream) {
    if (!h || !q || !out || !aligned16(q) || !aligned16(out)) return SEGKV_EINVAL;
    if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SEGKV_EINVAL;
    if (h->prompt_len < 0) return SEGKV_ESTATE;
    if (h->prompt_len + h->steps <= 0) return SEGKV_ESTATE;
    if (h->leader && h->leader->steps != h->steps) return SEGKV_ESTATE;   // the shared tables describe another step
    if (!tiled_supported(h->d)) return SEGKV_EINVAL;
    {
        int rc = ensure_lists(h, (cudaStream_t)stream);     // a kernel launch at most, never an allocation
        if (rc != SEGKV_OK) return rc;
    }
    const Tiling tl = choose_tiling(h, false);
    const int splits = tl.splits;
    SdpaArgs a = sdpa_args(h, q, out, alibi_slopes, splits);
    a.pdl = h->overlap;
    a.small = tl.small;
    a.one_wave = tl.one_wave;
    int too_big = 0;
    h->dbg_wait_ns = 0;
    h->dbg_skip = false;
    SEGKV_CUDA(launch_sdpa_tiled_static(h->d, a, tl.small ? h->tm_kp32 : h->tm_kp, tl.small ? h->tm_vp32 : h->tm_vp,
                                        tl.stages, (cudaStream_t)stream, &too_big));
    if (too_big) {
        snprintf(g_cuda_err, sizeof g_cuda_err,
                 "segkv_decode_sdpa_static: %d splits of this shape need more than the %zu bytes of built-in scratch",
                 splits, tiled_static_scratch_bytes());
        return SEGKV_ECAPACITY;
    }
    count_launch(h, (cudaStream_t)stream);
    return SEGKV_OK;
}

int segkv_decode_step(segkv_t h, int step, const int32_t* beam_parent, const void* k_new, const void* v_new,
                      const void* q, void* out, const float* alibi_slopes, void* stream) {
    if (!h || step < 0 || !k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return SEGKV_EINVAL;
    if (!q || !out || !aligned16(q) || !aligned16(out)) return SEGKV_EINVAL;
    if (step > 0 && (!beam_parent || (reinterpret_cast<uintptr_t>(beam_parent) & 3u))) return SEGKV_EINVAL;
    if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SEGKV_EINVAL;
    if (h->prompt_len < 0) return SEGKV_ESTATE;
    if (step != h->steps) return SEGKV_ESTATE;
    if (step >= h->d.max_steps) return SEGKV_ECAPACITY;
    if (!tiled_supported(h->d) || h->leader) {
        // shapes the tiled kernel does not take, and handles that use another handle's tables
        // (nothing to update in the attention kernel): the two separate launches
        int rc = segkv_append(h, step, beam_parent, k_new, v_new, stream);
        if (rc != SEGKV_OK) return rc;
        return segkv_decode_sdpa(h, q, out, alibi_slopes, stream);
    }
    const Dims& d = h->d;
    h->steps = step + 1;                 // the launch shape is chosen for the step being added
    const Tiling tl = choose_tiling(h, true);
    const int splits = tl.splits;
    const bool cluster = tl.cluster;
    h->steps = step;
    // rows a CTA's share of the steps can reach: beyond a tile and a half of them, deriving the rows
    // in the kernel costs more than the separate append launch (measured at prompts of 128 to 512
    // tokens with 128 steps: 10.0-10.6 us as two launches against 10.8-12.9 us fused)
    const long long rows_per_cta = (long long)((step + 1 + splits - 1) / splits) * d.beams;
    // (the small clustered form keeps a CTA's rows in one 32-row tile when the beams are few: exempt up to 4)
    const bool long_tail = h->splits_forced <= 0 && !(tl.small && tl.cluster && d.beams <= 4) &&                // a forced split count keeps the fused kernel
                           2 * rows_per_cta > 3 * tiled_tile_keys(d.head_dim, false);
    // a CTA with many prompt tiles to stream is bandwidth-bound and gains nothing from the fusion
    // (13B shape at batch 1: prompt 2048, 5 tiles per CTA, 12.3 us fused against 15.1 us as two
    // launches; prompt 4096, 10 tiles per CTA, 23.9 us against 22.0 us)
    const int tile_keys = tiled_tile_keys(d.head_dim, tl.small);
    const int ptiles_per_cta = ((h->prompt_len + tile_keys - 1) / tile_keys + splits - 1) / splits;
    const bool long_prompt = h->splits_forced <= 0 && ptiles_per_cta > 7;
    // (a launch of a few unsplit work groups is all latency: there the fused form saves a whole launch,
    // 3.7 against 6.0 us at the smallest evaluation shape)
    const bool fills_gpu = (long long)d.batch * d.kv_heads >= h->sm_count;
    if (((splits == 1 && fills_gpu) || long_tail || long_prompt) && !h->fuse_always) {
        // Work groups that fill the GPU on their own are bandwidth-bound: the separate append is
        // then ~1 % of the step and the list it makes keeps the response tiles dense and cheap
        // to build, so the two launches are the faster form.
        int rc = segkv_append(h, step, beam_parent, k_new, v_new, stream);
        if (rc != SEGKV_OK) return rc;
        return segkv_decode_sdpa(h, q, out, alibi_slopes, stream);
    }
    if (h->combine_forced == 2 && splits > 1 && !cluster) return SEGKV_EINVAL;
    if (!cluster && splits > h->ws_splits) {
        SEGKV_CUDA(cudaDeviceSynchronize());
        int rc = alloc_workspace(h, splits);
        if (rc != SEGKV_OK) return rc;
    }
    {
        int rc = ensure_chunk(h, step, (cudaStream_t)stream);
        if (rc != SEGKV_OK) return rc;
    }
    SdpaArgs a = sdpa_args(h, q, out, alibi_slopes, splits);
    a.steps = step + 1;
    a.anc = h->anc[(step + 1) & 1];      // table of step-1 (unused at step 0)
    a.cluster = cluster;
    a.small = tl.small;
    a.one_wave = tl.one_wave;
    // the first step after a prefill is fully serialised; from then on the prompt cannot change
    a.pdl = h->overlap && step > 0;
    a.prompt_immutable = step > 0;
    a.rows_immutable = step > 0 && rows_settled(h, (cudaStream_t)stream, false);
    a.fused = true;
    a.parent = step > 0 ? beam_parent : nullptr;
    a.k_new = k_new;
    a.v_new = v_new;
    a.kr_new_slab = k_slab_of(h, step);
    a.vr_new_slab = k_slab_of(h, step) + vdelta_of(h);
    a.anc_dst = h->anc[step & 1];
    a.parent_row = h->parent + (size_t)step * d.rows;
    h->dbg_wait_ns = 0;
    h->dbg_skip = false;
    SEGKV_CUDA(launch_sdpa_tiled(d, a, tl.small ? h->tm_kp32 : h->tm_kp, tl.small ? h->tm_vp32 : h->tm_vp, tl.stages,
                                 (cudaStream_t)stream));
    mark_written(h, &h->rows_mark, (cudaStream_t)stream);
    h->steps = step + 1;
    h->truncated = false;
    h->lists_valid = false;              // the fused kernel does not make the distinct-row lists
    return SEGKV_OK;
}

int segkv_step_host(segkv_t h, int step, const int32_t* beam_parent, const void* k_new, const void* v_new,
                    const void* q, void* out, const float* alibi_slopes, void* stream) {
    if (!h || !k_new || !v_new || !q || !out) return SEGKV_EINVAL;
    if (step > 0 && !beam_parent) return SEGKV_EINVAL;
    const Dims& d = h->d;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t qbytes = (size_t)d.rows * d.heads * d.head_dim * 2;
    const size_t kvbytes = (size_t)d.rows * d.kv_heads * d.head_dim * 2;
    if (step > 0)
        SEGKV_CUDA(cudaMemcpyAsync(h->st_parent, beam_parent, (size_t)d.rows * sizeof(int32_t),
                                   cudaMemcpyHostToDevice, st));
    SEGKV_CUDA(cudaMemcpyAsync(h->st_k, k_new, kvbytes, cudaMemcpyHostToDevice, st));
    SEGKV_CUDA(cudaMemcpyAsync(h->st_v, v_new, kvbytes, cudaMemcpyHostToDevice, st));
    SEGKV_CUDA(cudaMemcpyAsync(h->st_q, q, qbytes, cudaMemcpyHostToDevice, st));
    if (alibi_slopes)
        SEGKV_CUDA(cudaMemcpyAsync(h->st_slopes, alibi_slopes, (size_t)d.heads * sizeof(float),
                                   cudaMemcpyHostToDevice, st));
    int rc = segkv_decode_step(h, step, step > 0 ? h->st_parent : nullptr, h->st_k, h->st_v, h->st_q, h->st_out,
                               alibi_slopes ? h->st_slopes : nullptr, stream);
    if (rc != SEGKV_OK) return rc;
    SEGKV_CUDA(cudaMemcpyAsync(out, h->st_out, qbytes, cudaMemcpyDeviceToHost, st));
    SEGKV_CUDA(cudaStreamSynchronize(st));
    return SEGKV_OK;
}

size_t segkv_host_pack_bytes(segkv_t h, size_t* offsets) {
    if (!h) return 0;
    const Dims& d = h->d;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t qbytes = (size_t)d.rows * d.heads * d.head_dim * 2;
    const size_t kvbytes = (size_t)d.rows * d.kv_heads * d.head_dim * 2;
    size_t off[5];
    off[0] = 0;                                            // beam_parent  int32 [rows]
    off[1] = off[0] + up((size_t)d.rows * sizeof(int32_t));   // alibi slopes float [heads]
    off[2] = off[1] + up((size_t)d.heads * sizeof(float));    // k_new
    off[3] = off[2] + up(kvbytes);                            // v_new
    off[4] = off[3] + up(kvbytes);                            // q
    if (offsets)
        for (int i = 0; i < 5; ++i) offsets[i] = off[i];
    return off[4] + up(qbytes);
}

int segkv_step_host_packed(segkv_t h, int step, const void* host_in, void* host_out, int has_slopes, void* stream) {
    int rc = segkv_step_host_packed_async(h, step, host_in, host_out, has_slopes, stream);
    if (rc != SEGKV_OK) return rc;
    SEGKV_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    return SEGKV_OK;
}

int segkv_step_host_packed_async(segkv_t h, int step, const void* host_in, void* host_out, int has_slopes, void* stream) {
    if (!h || !host_in || !host_out) return SEGKV_EINVAL;
    const Dims& d = h->d;
    cudaStream_t st = (cudaStream_t)stream;
    size_t off[5];
    const size_t total = segkv_host_pack_bytes(h, off);
    const size_t qbytes = (size_t)d.rows * d.heads * d.head_dim * 2;
    SEGKV_CUDA(cudaMemcpyAsync(h->st_pack, host_in, total, cudaMemcpyHostToDevice, st));
    char* base = (char*)h->st_pack;
    int rc = segkv_decode_step(h, step, step > 0 ? (const int32_t*)(base + off[0]) : nullptr, base + off[2], base + off[3],
                               base + off[4], h->st_out, has_slopes ? (const float*)(base + off[1]) : nullptr, stream);
    if (rc != SEGKV_OK) return rc;
    SEGKV_CUDA(cudaMemcpyAsync(host_out, h->st_out, qbytes, cudaMemcpyDeviceToHost, st));
    return SEGKV_OK;
}

// Two streams of the library's own per device, for the copies of segkv_layers_step_host.
struct CopyStreams {
    cudaStream_t in, out;
    cudaEvent_t entry, done;
    bool ok;
};
CopyStreams* copy_streams(int dev) {
    static CopyStreams cs[64] = {};
    static std::mutex mu;
    if (dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lk(mu);
    CopyStreams& c = cs[dev];
    if (!c.ok) {
        if (cudaStreamCreateWithFlags(&c.in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&c.out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c.entry, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c.done, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        c.ok = true;
    }
    return &c;
}

int segkv_layers_step_host(const segkv_t* layers, int n, int step, const void* const* host_in, void* const* host_out,
                           int has_slopes, int redo, void* stream) {
    if (!layers || !host_in || !host_out || n <= 0) return SEGKV_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    for (int i = 0; i < n; ++i)
        if (!layers[i] || !layers[i]->ev_in || !layers[i]->ev_k) return SEGKV_EINVAL;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) cudaGetLastError();
    CopyStreams* cs = cap == cudaStreamCaptureStatusNone ? copy_streams(layers[0]->device) : nullptr;
    if (!cs) {
        // a stream being captured (or no streams to be had): everything in order on the caller's stream
        for (int i = 0; i < n; ++i) {
            segkv_t h = layers[i];
            if (redo && h->steps == step + 1 && !h->truncated) {
                h->steps -= 1;
                h->truncated = true;
            }
            const int rc = segkv_step_host_packed_async(h, step, host_in[i], host_out[i], has_slopes, stream);
            if (rc != SEGKV_OK) return rc;
        }
        return SEGKV_OK;
    }
    // Copies in on one stream, launches on the caller's, copies out on a third: layer i+1's inputs
    // travel while layer i computes and layer i-1's output travels back.  The copy-in stream starts
    // behind what the caller's stream holds now (the staging blocks may still be read by it), and the
    // caller's stream ends behind the last copy out, so waiting for it is waiting for everything.
    SEGKV_CUDA(cudaEventRecord(cs->entry, st));
    SEGKV_CUDA(cudaStreamWaitEvent(cs->in, cs->entry, 0));
    SEGKV_CUDA(cudaStreamWaitEvent(cs->out, cs->entry, 0));
    // When the caller's blocks of all layers lie back to back in host memory (one pinned array for the
    // stack), several layers travel in ONE copy each way: a copy call costs the host a few microseconds,
    // which at small shapes is as much as the layer's launch.  All inputs are queued first; the launches of
    // a group of layers wait for their group's copy, the group's outputs leave behind its last launch.
    {
        segkv_t h0 = layers[0];
        size_t off[5];
        const size_t total = segkv_host_pack_bytes(h0, off);
        const size_t qbytes = (size_t)h0->d.rows * h0->d.heads * h0->d.head_dim * 2;
        bool block = n >= 2;
        for (int i = 1; i < n && block; ++i) {
            const Dims &a = layers[i]->d, &b = h0->d;
            block = a.rows == b.rows && a.heads == b.heads && a.kv_heads == b.kv_heads && a.head_dim == b.head_dim &&
                    (const char*)host_in[i] == (const char*)host_in[0] + (size_t)i * total &&
                    (char*)host_out[i] == (char*)host_out[0] + (size_t)i * qbytes;
        }
        if (block) {
            if (h0->grp_in_cap < (size_t)n * total || h0->grp_out_cap < (size_t)n * qbytes) {
                // first call of this stack (or a longer one): the only allocation, outside the steady state
                SEGKV_CUDA(cudaDeviceSynchronize());
                if (h0->grp_in) cudaFree(h0->grp_in);
                if (h0->grp_out) cudaFree(h0->grp_out);
                h0->grp_in = h0->grp_out = nullptr;
                h0->grp_in_cap = h0->grp_out_cap = 0;
                SEGKV_CUDA(cudaMalloc(&h0->grp_in, (size_t)n * total));
                SEGKV_CUDA(cudaMalloc(&h0->grp_out, (size_t)n * qbytes));
                h0->grp_in_cap = (size_t)n * total;
                h0->grp_out_cap = (size_t)n * qbytes;
                SEGKV_CUDA(cudaEventRecord(cs->entry, st));
                SEGKV_CUDA(cudaStreamWaitEvent(cs->in, cs->entry, 0));
                SEGKV_CUDA(cudaStreamWaitEvent(cs->out, cs->entry, 0));
            }
            // groups of about 400 KB of input: long enough to amortise the call, short enough to start early
            int per = (int)((400u << 10) / (total ? total : 1));
            if (per < 1) per = 1;
            if (per > n) per = n;
            char* gin = (char*)h0->grp_in;
            char* gout = (char*)h0->grp_out;
            for (int g0 = 0; g0 < n; g0 += per) {
                const int cnt = n - g0 < per ? n - g0 : per;
                SEGKV_CUDA(cudaMemcpyAsync(gin + (size_t)g0 * total, host_in[g0], (size_t)cnt * total, cudaMemcpyHostToDevice, cs->in));
                SEGKV_CUDA(cudaEventRecord(layers[g0]->ev_in, cs->in));
            }
            for (int g0 = 0; g0 < n; g0 += per) {
                const int cnt = n - g0 < per ? n - g0 : per;
                SEGKV_CUDA(cudaStreamWaitEvent(st, layers[g0]->ev_in, 0));
                for (int i = g0; i < g0 + cnt; ++i) {
                    segkv_t h = layers[i];
                    if (redo && h->steps == step + 1 && !h->truncated) {
                        h->steps -= 1;
                        h->truncated = true;
                    }
                    char* base = gin + (size_t)i * total;
                    const int rc = segkv_decode_step(h, step, step > 0 ? (const int32_t*)(base + off[0]) : nullptr, base + off[2],
                                                     base + off[3], base + off[4], gout + (size_t)i * qbytes,
                                                     has_slopes ? (const float*)(base + off[1]) : nullptr, stream);
                    if (rc != SEGKV_OK) return rc;
                }
                SEGKV_CUDA(cudaEventRecord(layers[g0]->ev_k, st));
                SEGKV_CUDA(cudaStreamWaitEvent(cs->out, layers[g0]->ev_k, 0));
                SEGKV_CUDA(cudaMemcpyAsync(host_out[g0], gout + (size_t)g0 * qbytes, (size_t)cnt * qbytes, cudaMemcpyDeviceToHost, cs->out));
            }
            SEGKV_CUDA(cudaEventRecord(cs->done, cs->out));
            SEGKV_CUDA(cudaStreamWaitEvent(st, cs->done, 0));
            return SEGKV_OK;
        }
    }
    for (int i = 0; i < n; ++i) {
        segkv_t h = layers[i];
        if (redo && h->steps == step + 1 && !h->truncated) {
            h->steps -= 1;
            h->truncated = true;
        }
        const Dims& d = h->d;
        size_t off[5];
        const size_t total = segkv_host_pack_bytes(h, off);
        const size_t qbytes = (size_t)d.rows * d.heads * d.head_dim * 2;
        SEGKV_CUDA(cudaMemcpyAsync(h->st_pack, host_in[i], total, cudaMemcpyHostToDevice, cs->in));
        SEGKV_CUDA(cudaEventRecord(h->ev_in, cs->in));
        SEGKV_CUDA(cudaStreamWaitEvent(st, h->ev_in, 0));
        char* base = (char*)h->st_pack;
        const int rc = segkv_decode_step(h, step, step > 0 ? (const int32_t*)(base + off[0]) : nullptr, base + off[2],
                                         base + off[3], base + off[4], h->st_out,
                                         has_slopes ? (const float*)(base + off[1]) : nullptr, stream);
        if (rc != SEGKV_OK) return rc;
        SEGKV_CUDA(cudaEventRecord(h->ev_k, st));
        SEGKV_CUDA(cudaStreamWaitEvent(cs->out, h->ev_k, 0));
        SEGKV_CUDA(cudaMemcpyAsync(host_out[i], h->st_out, qbytes, cudaMemcpyDeviceToHost, cs->out));
    }
    SEGKV_CUDA(cudaEventRecord(cs->done, cs->out));
    SEGKV_CUDA(cudaStreamWaitEvent(st, cs->done, 0));
    return SEGKV_OK;
}

int segkv_reset(segkv_t h, int keep_prompt) {
    if (!h) return SEGKV_EINVAL;
    h->steps = 0;
    h->truncated = false;
    if (!keep_prompt) {
        h->prompt_len = -1;
        h->tm_valid = false;
    }
    return SEGKV_OK;
}

int segkv_truncate_last(segkv_t h) {
    if (!h) return SEGKV_EINVAL;
    if (h->steps <= 0 || h->truncated) return SEGKV_ESTATE;
    h->steps -= 1;
    h->truncated = true;
    return SEGKV_OK;
}

int segkv_get_ancestry(segkv_t h, int32_t* host_out, void* stream) {
    if (!h || !host_out) return SEGKV_EINVAL;
    if (h->truncated) return SEGKV_ESTATE;   // the table of the dropped step is what is stored
    if (h->steps == 0) return SEGKV_OK;
    const Dims& d = h->d;
    if (h->leader && h->leader->steps != h->steps) return SEGKV_ESTATE;
    const int32_t* src = index_of(h)->anc[(h->steps - 1) & 1];
    SEGKV_CUDA(cudaMemcpy2DAsync(host_out, (size_t)h->steps * sizeof(int32_t), src,
                                 (size_t)d.max_steps * sizeof(int32_t), (size_t)h->steps * sizeof(int32_t),
                                 d.rows, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    SEGKV_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    return SEGKV_OK;
}

int segkv_get_unique_rows(segkv_t h, int32_t* host_out, void* stream) {
    if (!h || !host_out) return SEGKV_EINVAL;
    if (h->truncated) return SEGKV_ESTATE;
    const Dims& d = h->d;
    memset(host_out, 0, (size_t)d.batch * sizeof(int32_t));
    if (h->steps == 0) return SEGKV_OK;
    // count on the host what the attention kernel de-duplicates on the fly
    int32_t* anc = (int32_t*)malloc((size_t)d.rows * h->steps * sizeof(int32_t));
    if (!anc) return SEGKV_ENOMEM;
    int rc = segkv_get_ancestry(h, anc, stream);
    if (rc == SEGKV_OK) {
        for (int b = 0; b < d.batch; ++b) {
            int n = 0;
            for (int s = 0; s < h->steps; ++s)
                for (int j = 0; j < d.beams; ++j) {
                    bool first = true;
                    const int32_t rj = anc[(size_t)(b * d.beams + j) * h->steps + s];
                    for (int i = 0; i < j && first; ++i)
                        first = anc[(size_t)(b * d.beams + i) * h->steps + s] != rj;
                    n += first ? 1 : 0;
                }
            host_out[b] = n;
        }
    }
    free(anc);
    return rc;
}

int segkv_get_error(segkv_t h, int* device_flags) {
    if (!h || !device_flags) return SEGKV_EINVAL;
    SEGKV_CUDA(cudaDeviceSynchronize());
    SEGKV_CUDA(cudaMemcpy(device_flags, h->err_word, sizeof(int), cudaMemcpyDeviceToHost));
    SEGKV_CUDA(cudaMemset(h->err_word, 0, sizeof(int)));
    return SEGKV_OK;
}

int segkv_steps(segkv_t h) { return h ? h->steps : SEGKV_EINVAL; }
int segkv_prompt_len(segkv_t h) { return h ? h->prompt_len : SEGKV_EINVAL; }

int segkv_set_tuning(segkv_t h, int splits, int stages, int combine) {
    if (!h || splits < 0 || splits > kMaxSplits || stages < 0 || stages > 16) return SEGKV_EINVAL;
    if (combine < 0 || combine > 2) return SEGKV_EINVAL;
    if (stages > 0 && tiled_smem_bytes(h->d, stages, h->tile_forced == 32) > h->smem_optin) return SEGKV_EINVAL;
    if (splits > h->ws_splits) {
        // a forced split count beyond what the handle was sized for: grow the workspace here, not in the decode loop
        SEGKV_CUDA(cudaDeviceSynchronize());
        int rc = alloc_workspace(h, splits);
        if (rc != SEGKV_OK) return rc;
    }
    h->splits_forced = splits;
    h->stages_forced = stages;
    h->combine_forced = combine;
    h->fuse_always = splits == 1;        // an explicit single split still exercises the fused kernel
    return SEGKV_OK;
}

int segkv_get_splits(segkv_t h) {
    if (!h) return SEGKV_EINVAL;
    if (!tiled_supported(h->d)) return 1;
    return choose_tiling(h, false).splits;
}

int segkv_decode_sdpa_rowwise(segkv_t h, const void* q, void* out, const float* alibi_slopes, void* stream) {
    if (!h || !q || !out || !aligned16(q) || !aligned16(out)) return SEGKV_EINVAL;
    if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SEGKV_EINVAL;
    if (h->prompt_len < 0) return SEGKV_ESTATE;
    if (h->prompt_len + h->steps <= 0) return SEGKV_ESTATE;
    SdpaArgs a = sdpa_args(h, q, out, alibi_slopes, 1);
    SEGKV_CUDA(launch_sdpa_rowwise(h->d, a, (cudaStream_t)stream));
    count_launch(h, (cudaStream_t)stream);
    return SEGKV_OK;
}

int segkv_set_overlap(segkv_t h, int enable) {
    if (!h) return SEGKV_EINVAL;
    h->overlap = enable != 0;
    return SEGKV_OK;
}

int segkv_share_index(segkv_t h, segkv_t leader) {
    if (!h || h == leader) return SEGKV_EINVAL;
    if (h->steps != 0) return SEGKV_ESTATE;
    if (leader) {
        if (leader->leader) return SEGKV_EINVAL;             // a follower cannot lead
        const Dims &a = h->d, &b = leader->d;
        if (a.batch != b.batch || a.beams != b.beams || a.max_steps != b.max_steps) return SEGKV_EINVAL;
        if (leader->steps != 0) return SEGKV_ESTATE;
        if (h->followers > 0) return SEGKV_EINVAL;           // a handle that leads cannot follow
    }
    if (h->leader) h->leader->followers--;
    if (leader) leader->followers++;
    h->leader = leader;
    return SEGKV_OK;
}

int segkv_set_prompt_layout(segkv_t h, int layout) {
    if (!h || layout < SEGKV_PROMPT_HEAD_MAJOR || layout > SEGKV_PROMPT_SEQ_FIRST) return SEGKV_EINVAL;
    if (h->prompt_len >= 0) return SEGKV_ESTATE;     // a prompt is stored in the current layout
    h->d.prompt_layout = layout;
    return SEGKV_OK;
}

int segkv_set_prefill_tuning(segkv_t h, int row_groups) {
    if (!h || row_groups < 0 || row_groups > 2) return SEGKV_EINVAL;
    h->prefill_groups = row_groups;
    return SEGKV_OK;
}

int segkv_set_tile(segkv_t h, int tile_keys) {
    if (!h || (tile_keys != 0 && tile_keys != 32 && tile_keys != 64)) return SEGKV_EINVAL;
    if (tile_keys == 32 && !tiled_small_ok(h->d)) return SEGKV_EINVAL;
    h->tile_forced = tile_keys;
    return SEGKV_OK;
}

int segkv_set_persistent(segkv_t h, int mode) {
    if (!h || mode < -1 || mode > 1) return SEGKV_EINVAL;
    if (mode == 1 && !stream_supported(h->d)) return SEGKV_EINVAL;
    h->persist_mode = mode;
    return SEGKV_OK;
}

int segkv_read_bandwidth(const void* dev_buf, size_t bytes, int repeats, float* gbs_out, void* stream) {
    if (!dev_buf || !gbs_out || bytes < 16 || repeats <= 0 || !aligned16(dev_buf)) return SEGKV_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    SEGKV_CUDA(cudaGetDevice(&dev));
    SEGKV_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    unsigned* sink = nullptr;
    SEGKV_CUDA(cudaMalloc((void**)&sink, 64 * sizeof(unsigned)));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaMemsetAsync(sink, 0, 64 * sizeof(unsigned), st);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    for (int i = 0; i < 3 && e == cudaSuccess; ++i) e = launch_read_stream(dev_buf, bytes, sink, sms, st);   // warm-up
    if (e == cudaSuccess) e = cudaEventRecord(e0, st);
    for (int i = 0; i < repeats && e == cudaSuccess; ++i) e = launch_read_stream(dev_buf, bytes, sink, sms, st);
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    if (e != cudaSuccess) return cuda_fail(e, "segkv_read_bandwidth");
    *gbs_out = (float)((double)bytes * repeats / (ms * 1e-3) / 1e9);
    return SEGKV_OK;
}

int segkv_debug_inject(segkv_t h, long long wait_limit_ns, int skip_arrival) {
    if (!h || wait_limit_ns < 0) return SEGKV_EINVAL;
    h->dbg_wait_ns = (unsigned long long)wait_limit_ns;
    h->dbg_skip = skip_arrival != 0;
    return SEGKV_OK;
}

long long segkv_launch_count(segkv_t h) { return h ? h->launches : (long long)SEGKV_EINVAL; }

}  // extern "C"
