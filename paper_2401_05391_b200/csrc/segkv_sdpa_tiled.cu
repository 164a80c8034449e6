// Tiled split-KV decode attention for sm_100a.
//
// What it computes: paper Section 3.3 ("Customized SDPA Kernel") — for each
// (request, kv head) work group the query block Q[BW, D] attends to the shared
// prompt K/V [N_prompt, D] and to the index-selected response rows, with one
// softmax over both parts.  How it is organised here is specific to B200:
//
//  * grid = (request, kv head, split).  A CTA owns ALL beams (and all query
//    heads of the kv head's group) of its work group, so a K/V byte staged in
//    shared memory is used by every beam: prompt bytes cross HBM once per
//    request, not once per beam (the saving Section 4.2.1 describes).
//  * two producer warps feed a ring of shared-memory stages.  The TMA warp
//    fetches prompt tiles (cp.async.bulk.tensor, 128-byte swizzle) from the
//    head-major prompt segment; it sets the mbarriers up itself and issues the
//    first ring before the CTA has synchronised.  The gather warp copies
//    response rows one by one with 16-byte cp.async (16 lanes per 256-byte
//    row) into the same swizzled layout: the index select of Section 3.3
//    folded into the load.  Every row carries its step and the set of beams
//    that read it; scores of other beams are masked, so a row shared by
//    several beams is fetched once.
//      - separate form (segkv_decode_sdpa): the rows come from the request's
//        list of DISTINCT rows that the append kernel made;
//      - fused form (segkv_decode_step, template FUSED): one lane per (step,
//        beam) reads the previous step's beam-index table, resolves the new
//        parents with a shuffle (anc_t[j][s] = anc_{t-1}[parent[j]][s]),
//        removes duplicates among the lanes of a step, packs the distinct rows
//        with a warp prefix sum, stores the new table column, and takes the
//        new step's rows straight from the caller's k_new / v_new.
//  * consumer warps take 16 keys of a tile each.  Scores are a small GEMM on
//    tensor cores with the KEYS on the M side: S^T[16 keys, 8 cols] = K . Q^T
//    (mma.sync m16n8k16, fp32 accumulate), so the BW=4 beams pad only to 8.
//    Online softmax in fp32 (base-2 exponent), P^T transposed in registers
//    (movmatrix) and O^T[16 d, 8 cols] += V^T . P^T, V^T read with
//    ldmatrix.trans.  Each warp keeps its own running max / sum / O^T.
//  * epilogue: warps merge through shared memory; with more than one split the
//    partial (m, l, O) goes to a global workspace and the last CTA of the work
//    group to arrive (acq_rel ticket, nobody waits) folds the splits in one
//    pass, or, on request, the splits form a thread-block cluster and exchange
//    slices of the (column, d) plane through distributed shared memory.
//  * programmatic dependent launch: prompt tiles are requested before the
//    previous kernel of the stream has finished (nothing in a decode loop
//    writes the prompt segment); everything else follows griddepcontrol.wait,
//    and dependents are released only after that wait.
//
// All mbarrier waits are bounded: on expiry the kernel sets
// SEGKV_DEV_WAIT_LIMIT in the error word and winds down.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "segkv_internal.h"
#include "segkv_ptx.cuh"

namespace segkv_impl {

namespace {

using namespace ptx;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive_relaxed() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Store to another CTA of the cluster that reports its bytes to an mbarrier of that CTA: the
// receiver learns of the data by waiting on its own barrier, nobody meets at a cluster barrier.
__device__ __forceinline__ void st_async_v4(uint32_t addr, float4 v, uint32_t mbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1,%2,%3,%4}, [%5];"
                 ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(mbar) : "memory");
}
__device__ __forceinline__ void st_async_v2(uint32_t addr, float a, float b, uint32_t mbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1,%2}, [%3];"
                 ::"r"(addr), "f"(a), "f"(b), "r"(mbar) : "memory");
}
// Bounded wait on an mbarrier of this CTA whose phase is completed by other CTAs' stores.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    const uint64_t t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 1024; ++i) {
            uint32_t ok;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
            if (ok) return true;
        }
        if (global_ns() - t0 > limit_ns) return false;
    }
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Programmatic dependent launch: let the next kernel of the stream begin, and wait for the
// previous one to have completed with its writes visible (no-ops without the launch attribute).
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

#ifdef SEGKV_TIMELINE
}  // namespace
__device__ unsigned long long g_timeline[8 * 512 * 32];   // per CTA: 16 x %globaltimer, then 16 x clock64
#define SEGKV_CLK(ev, cond)                                                                \
    do {                                                                                   \
        if ((cond) && (threadIdx.x & 31) == 0 && blockIdx.x < 512) {                       \
            g_timeline[((p.dbg_launch & 7) * 512 + blockIdx.x) * 32 + 16 + (ev)] = (unsigned long long)clock64(); \
        }                                                                                  \
    } while (0)
#define SEGKV_STAMP(ev)                                                                    \
    do {                                                                                   \
        if ((threadIdx.x & 31) == 0 && blockIdx.x < 512) {                                 \
            if ((ev) == 0) g_timeline[((p.dbg_launch & 7) * 512 + blockIdx.x) * 32] = global_ns(); \
            g_timeline[((p.dbg_launch & 7) * 512 + blockIdx.x) * 32 + 16 + (ev)] = (unsigned long long)clock64(); \
        }                                                                                  \
    } while (0)
namespace {
#else
#define SEGKV_CLK(ev, cond) do {} while (0)
#define SEGKV_STAMP(ev) do {} while (0)
#endif

// A CTA whose bounded wait ran out adds this to its work group's arrival counter on top of its
// ticket (splits are at most kMaxSplits, far below it).
constexpr int kTicketAborted = 1 << 16;

template <int N> struct IntC { static constexpr int value = N; };

struct TiledParams {
    const void* q;
    void* out;
    const float* slopes;
    const char* kr;          // response K, fixed capacity (V row = K row + vdelta)
    const char* const* k_chunks;   // growing capacity: chunk base pointers, chunk_steps steps each
    long long vdelta;
    const URow* ulist;
    const int32_t* ucount;
    const int32_t* plens;    // per-request prompt lengths, or NULL: every request has P tokens
    float* ws_o;    // [slab][S][ncols][D]   un-normalised partial outputs (ticket combine only)
    float* ws_ml;   // [slab][S][ncols][2]   running max (base-2 domain) and sum
    int* tickets;
    int* err_word;
    // fused decode step only: the step's inputs and the cache locations they are stored to
    const int32_t* anc_prev; // beam-index table of the previous step
    const int32_t* parent;   // [rows] beam parents of the new step (NULL at step 0)
    const char* k_new;       // [rows, Hkv, D]
    const char* v_new;
    char* kr_new_slab;       // slab of the new step inside the response segment
    char* vr_new_slab;
    int32_t* anc_dst;        // table of the new step
    int32_t* parent_row;     // row of the parent table
    int fused;      // 1: steps-1 is a new step whose rows come from k_new / v_new and whose beam-index
                    //    column is derived here from `parent` and the previous table
    int P, steps, S, W, G, H, Hkv, rows, max_steps, ncols, stages;
    int chunk_steps;   // 0: the response segment is one array
    int quota;      // distinct response rows per split (the last split also takes any excess)
    int tail_groups;   // the last tail_groups work groups are cut into tail_S splits instead of S (a ragged last
    int tail_S;        // wave spread over all SMs); their quota is tail_quota; the split workspace holds only
    int tail_quota;    // the items from ws_item0 on
    int ws_item0;
    int head_items;    // CTAs of the work groups before the tail
    int cluster;    // 1: the S CTAs of a work group form a thread-block cluster
    int early_prompt;  // 1: prompt tiles may be fetched before the previous kernel has completed
    int early_rows;    // 1: so may the response rows of earlier steps and (separate form) the row lists
    int resv;          // 1: the last stage is set aside for the CTA's first response tile (see the kernel)
    int one_wave;      // 1: all CTAs of the launch are resident at once (what cannot be fetched yet is asked into the L2)
    int dbg_skip;      // test aid: the gather warp leaves out one plain barrier arrival, so that a wait runs out
    unsigned long long wait_ns;   // limit of every bounded wait
#ifdef SEGKV_TIMELINE
    int dbg_launch;
#endif
    float scale2;   // log2(e) / sqrt(D)
};

// Shared-memory carve-up (after rounding the base up to 1024 bytes):
//   stages x { K tile, V tile }      each tile = D/64 boxes of [TILE rows][128 B], 128B-swizzled
//   stages x URow[TILE]              per-key row id and beam mask of response tiles
//     (the warp-merge buffer and the ticket-combine scratch of the epilogue re-use this area)
//   full[stages], empty[stages], hand   mbarriers
//   recv_o, recv_ml                  landing area for the other CTAs' partials (cluster combine)
template <int D, int CW>
struct Layout {
    static constexpr int TILE = 16 * CW;
    static constexpr int BOX_BYTES = TILE * 128;
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int META_BYTES = TILE * (int)sizeof(URow);
    static __host__ __device__ constexpr size_t body(int stages, int nt) {
        size_t ring = (size_t)stages * (STAGE_BYTES + META_BYTES);
        size_t merge = (size_t)CW * 8 * nt * (D + 4 + 2) * 4;
        size_t comb = (size_t)2 * kMaxSplits * 8 * nt * 4;
        size_t b = ring > merge ? ring : merge;
        b = b > comb ? b : comb;
        return (b + 127) & ~(size_t)127;
    }
    static __host__ __device__ constexpr size_t bars(int stages) {
        // mbarriers, per-stage {count, last} of response tiles, then the gather warp's row pointers
        return (((size_t)stages * 24 + 16 + 127) & ~(size_t)127) + (size_t)TILE * 16;
    }
    static __host__ __device__ constexpr size_t recv(int nt) {
        return (size_t)8 * nt * D * 4 + (size_t)kMaxCluster * 8 * nt * 2 * 4;
    }
    static __host__ __device__ constexpr size_t bytes(int stages, int nt) {
        return 1024 + body(stages, nt) + bars(stages) + recv(nt);
    }
};

template <typename T, int D, int NT, int CW, bool FUSED>
__global__ void __launch_bounds__(32 * (CW + 2), NT > 1 ? 1 : (CW == 2 && D <= 128 ? 4 : 2))
sdpa_tiled_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const TiledParams p) {
    using L = Layout<D, CW>;
    constexpr int TILE = L::TILE;
    constexpr int KS = D / 16;           // k-steps of Q.K, m-tiles of P.V
    constexpr int NTHREADS = 32 * (CW + 2);
    constexpr int DP = D + 4;            // padded row of the merge buffer (conflict-free)
    constexpr int UK = (TILE + 31) / 32;
    constexpr int D4 = D / 4;
    constexpr int TMA_WARP = CW, GATHER_WARP = CW + 1;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stages = p.stages;
    uint8_t* ring = smem;
    URow* meta = reinterpret_cast<URow*>(ring + (size_t)stages * L::STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::body(stages, NT));
    float* recv_o = reinterpret_cast<float*>(smem + L::body(stages, NT) + L::bars(stages));   // [S][slice]
    float* recv_ml = recv_o + 8 * NT * D;                                                     // [S][ncols][2]
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + stages), hand = smem_u32(bars + 2 * stages);
    int2* tile_hdr = reinterpret_cast<int2*>(bars + 2 * stages + 1);                           // [stages] {count, last}
    const uint32_t recvbar = smem_u32(bars + 3 * stages + 1);          // cluster merge: the other CTAs' partials have landed
    const char** gk = reinterpret_cast<const char**>(reinterpret_cast<uint8_t*>(recv_o) - (size_t)TILE * 16);  // [TILE] K row pointers
    const char** gv = gk + TILE;                                                               // [TILE] V row pointers
    __shared__ int s_last, s_abort;

    // When the response rows may be fetched ahead of the grid-dependency wait, the LAST stage is set
    // aside for the CTA's first response tile (usually its only one): the long chain of its fetch
    // (count or table -> addresses -> copies) is then over before the wait returns, whatever the
    // prompt tiles do with the other RS stages, which they share as a ring.  Further response tiles
    // follow the prompt tiles through that ring.  The order in which tiles are CONSUMED never
    // changes (prompt, then response), so results do not depend on which way a launch was made.
    const int RS = stages - p.resv;
    const int rstage = stages - 1;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) SEGKV_STAMP(0);
    // blockIdx -> (work group, split): S splits per group, except that the last tail_groups groups have tail_S
    const int head_items = p.head_items;
    const bool in_tail = (int)blockIdx.x >= head_items;
    const int SS = in_tail ? p.tail_S : p.S;                         // splits of THIS work group
    const int quota = in_tail ? p.tail_quota : p.quota;
    const int split = in_tail ? ((int)blockIdx.x - head_items) % p.tail_S : (int)blockIdx.x % p.S;
    const int slab = in_tail ? head_items / p.S + ((int)blockIdx.x - head_items) / p.tail_S
                             : (int)blockIdx.x / p.S;                // b * Hkv + kvh
    const int ws_item = (int)blockIdx.x - p.ws_item0;               // this CTA's place in the split workspace
    const int b = slab / p.Hkv, kvh = slab % p.Hkv;

    // This CTA's share of the work group: whole prompt tiles (known from the launch shape
    // alone, so their loads start at once) and a range of the request's distinct response
    // rows (known once the row count has been read).
    // prompt length of this request: the launch's, or its own when the prompts are ragged (rows
    // between the two hold zeros); written at prefill time, so it may be read before the
    // grid-dependency wait
    const int P = p.plens ? __ldg(p.plens + b) : p.P;
    const int ntp = (P + TILE - 1) / TILE;
    const int pt0 = (int)((long long)split * ntp / SS), pt1 = (int)((long long)(split + 1) * ntp / SS);
    const int npt = pt1 - pt0;
    const URow* ulist_b = p.ulist + (size_t)b * p.W * p.max_steps;
    // fused step: response steps are cut evenly over the splits (known from the launch shape alone)
    const int rs0 = (int)((long long)split * p.steps / SS), rs1 = (int)((long long)(split + 1) * p.steps / SS);

    auto issue_prompt_tile = [&](int k, int st) {
        const uint32_t full = full0 + 8 * st;
        if (lane == 0) {
            const uint32_t k_dst = smem_u32(ring + (size_t)st * L::STAGE_BYTES);
            const uint32_t v_dst = k_dst + L::TILE_BYTES;
            mbar_arrive_expect_tx(full, (uint32_t)L::STAGE_BYTES);
            const int y = (pt0 + k) * TILE;
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx) {
                tma_load_4d(k_dst + bx * L::BOX_BYTES, &tm_k, bx * 64, kvh, y, b, full);
                tma_load_4d(v_dst + bx * L::BOX_BYTES, &tm_v, bx * 64, kvh, y, b, full);
            }
        }
        mbar_arrive(full);      // lanes 1..31, and lane 0 a second time (the count is the gather warp's)
    };

    int tma_issued = 0;       // TMA warp: fills started (for the wind-down after an expired wait)
    if (warp == TMA_WARP) {
        // The warp that issues the bulk loads sets the barriers up itself and starts the
        // first round of prompt tiles before the rest of the CTA has even synchronised.
        if (lane == 0) {
            for (int s = 0; s < stages; ++s) {
                mbar_init(full0 + 8 * s, 33);     // every lane of the filling warp, plus lane 0 once more
                mbar_init(empty0 + 8 * s, CW);    // one arrival per consumer warp
            }
            mbar_init(hand, 1);                   // ring handed from the TMA warp to the gather warp
            if (p.cluster) {
                // the S partials of this CTA's slice of the (column, d) plane and S x ncols {max, sum} pairs
                mbar_init(recvbar, 1);
                mbar_arrive_expect_tx(recvbar, (uint32_t)(p.ncols * D * 4 + p.S * p.ncols * 8));
            }
            s_abort = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            fence_proxy_async();
            if (npt > 0) {
                prefetch_tmap(&tm_k);
                prefetch_tmap(&tm_v);
            }
        }
        __syncwarp();
        // The prompt segment does not change during decoding, so when the host says so its
        // tiles are requested before the previous kernel of the stream has finished.
        if (!p.early_prompt) grid_wait();
        const int first = min(npt, RS);
        for (int k = 0; k < first; ++k) issue_prompt_tile(k, k);
        tma_issued = first;
        if (first == npt && lane == 0) mbar_arrive(hand);
        // Prompt tiles that have to wait for a stage of the ring are at least brought into the L2,
        // so that their turn costs an L2 hit, not an HBM round trip, after the wait (7.2 -> 6.5 us for the
        // separate call at the Llama2-7B shape).  Not in the small form of the fused step: it has its
        // reserved response tile to consume while those tiles travel and was measured a little faster
        // without the extra traffic ahead of its predecessor's last loads, 7.55 against 7.61 us.
        constexpr bool kEarlyResp = FUSED && CW == 2 && D <= 128 && NT == 1;     // the fused small form
        if (!kEarlyResp && p.early_prompt && p.one_wave && lane == 0) {       // (a launch of several waves is bound by bandwidth: no fetching ahead of need)
            for (int k = first; k < npt; ++k) {
                const int y = (pt0 + k) * TILE;
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx) {
                    tma_prefetch_4d(&tm_k, bx * 64, kvh, y, b);
                    tma_prefetch_4d(&tm_v, bx * 64, kvh, y, b);
                }
            }
        }
        SEGKV_STAMP(3);
    } else if (warp == 0) {
        // The query rows are written by the kernel before this one, so they may only be READ after
        // the wait; asking the L2 for their lines is harmless before it (a line fetched early is
        // overwritten in place by the producer), and the read after the wait then finds them there.
        constexpr int LPR = D * 2 / 128;                         // 128-byte lines per query row
        for (int i = lane; i < p.ncols * LPR; i += 32) {
            const int col = i / LPR;
            const char* qrow = reinterpret_cast<const char*>(p.q) +
                               ((size_t)(b * p.W + col / p.G) * p.H + kvh * p.G + col % p.G) * (size_t)(D * 2);
            prefetch_l2(qrow + (i % LPR) * 128);
        }
    }
    // Consumer warps: what needs no data of the previous kernel (addresses, column masks) is worked
    // out before the wait, so that the query loads go out the moment it returns.
    const T* qrow_c[NT];
    const float* slope_c[NT][2];
    uint32_t beambit[NT][2];
    if (warp < CW) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int col = nt * 8 + (lane >> 2);             // Q^T as the B operand: this lane holds column lane/4
            const bool cv = col < p.ncols;
            const int j = cv ? col / p.G : 0, hg = cv ? col % p.G : 0;
            qrow_c[nt] = cv ? reinterpret_cast<const T*>(p.q) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D : nullptr;
#pragma unroll
            for (int c = 0; c < 2; ++c) {                     // the two score columns this lane owns
                const int col2 = nt * 8 + (lane & 3) * 2 + c;
                const bool cv2 = col2 < p.ncols;
                beambit[nt][c] = cv2 ? (1u << (col2 / p.G)) : 0u;
                slope_c[nt][c] = (cv2 && p.slopes) ? p.slopes + kvh * p.G + col2 % p.G : nullptr;
            }
        }
    }
    if (p.cluster) cluster_arrive_relaxed();     // "this CTA has started" (waited for before any remote store)
    __syncthreads();
    // Everything else (q, row lists, parents, response rows, outputs) follows the previous kernel.
    // The next kernel is let go only after this wait, so a kernel that starts early behind this
    // one finds every kernel before this one's predecessor complete.  (The gather warp, when the
    // host vouches for its inputs, works ahead and waits later.)
    const bool gather_ahead = warp == GATHER_WARP && p.early_rows;
    // Consumer warps of a launch that starts early have nothing to do before the wait; they spend the
    // time running one tile's worth of their loop on whatever the first stage holds and throwing the
    // result away: the loop's instructions are then in the instruction cache when the real first
    // tile comes (straight-line code that runs once per CTA is bound by instruction fetch).
    const bool cons_ahead = warp < CW && p.early_prompt;
    // (Warps that work ahead wait later and leave the release to the others: the TMA warp always comes
    // through here, and one thread's release stands for its CTA.)
    if (!gather_ahead && !cons_ahead) {
        grid_wait();
        grid_launch_dependents();
    }
    if (tid == 0 && !cons_ahead) SEGKV_STAMP(2);

    // consumer state (declared here so that the epilogue sees it)
    float o_acc[NT][KS][4];
    float m_run[NT][2], l_run[NT][2];
    bool cons_ok = true;          // this consumer warp has seen all of its tiles

    if (warp == TMA_WARP) {
        // ============================ prompt tiles beyond the first round ============================
        bool ok = true;
        for (int k = tma_issued; k < npt; ++k) {
            const int st = k % RS;
            ok = mbar_wait(empty0 + 8 * st, (((uint32_t)(k / RS)) & 1) ^ 1, p.wait_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            issue_prompt_tile(k, st);
            tma_issued = k + 1;
            if (k + 1 == npt && lane == 0) mbar_arrive(hand);
        }
        if (!ok && lane == 0) {
            atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            s_abort = 1;
        }
    } else if (warp == GATHER_WARP) {
        // ================== response tiles: index select fused into the load ==================
        // A tile holds up to TILE distinct response rows of the request, each with its step and
        // the set of beams that read it (rows shared by several beams are fetched once).  The
        // ring is taken over from the TMA warp only when the last prompt tile has been issued
        // (a parity wait cannot tell a far-future round of a stage from the current one).
        constexpr int CPR = D / 8;        // 16-byte chunks per row
        constexpr int RPI = 32 / CPR;     // rows covered by one warp-wide copy
        const size_t slab_bytes = (size_t)p.rows * p.Hkv * (size_t)(D * 2);
        // K slab of response step s: in the one array, or in the chunk that holds the step
        auto k_slab = [&](int s) -> const char* {
            if (p.chunk_steps == 0) return p.kr + (size_t)s * slab_bytes;
            const int c = s / p.chunk_steps;
            return p.k_chunks[c] + (size_t)(s - c * p.chunk_steps) * slab_bytes;
        };
        // Copy rows [0, cnt) of the tile whose row pointers (gk, gv) have been written.  One
        // warp-wide copy moves whole rows (CPR lanes per row): fully coalesced.  The arrival on
        // the stage's full barrier fires when this lane's copies have landed.
        auto copy_rows = [&](int st, int from, int cnt, bool arrive) {
            const uint32_t full = full0 + 8 * st;
            const uint32_t k_dst = smem_u32(ring + (size_t)st * L::STAGE_BYTES), v_dst = k_dst + L::TILE_BYTES;
            const int c = lane % CPR;
            const uint32_t c_off = (uint32_t)(c / 8) * L::BOX_BYTES;
            __syncwarp();                              // gk / gv written by other lanes
#pragma unroll
            for (int i = 0; i < TILE / RPI; ++i) {
                if (i * RPI < cnt && (i + 1) * RPI > from) {      // warp-uniform
                    const int key = i * RPI + lane / CPR;
                    if (key < cnt && key >= from) {
                        const uint32_t off = c_off + (uint32_t)key * 128 + (uint32_t)(((c & 7) ^ (key & 7)) << 4);
                        if constexpr (FUSED) {             // rows may sit in the caller's k_new / v_new
                            cp_async_16(k_dst + off, gk[key] + c * 16);
                            cp_async_16(v_dst + off, gv[key] + c * 16);
                        } else {                           // a V row sits a constant behind its K row
                            const char* src = gk[key] + c * 16;
                            cp_async_16(k_dst + off, src);
                            cp_async_16(v_dst + off, src + p.vdelta);
                        }
                    }
                }
            }
            if (arrive) cp_async_mbar_arrive_noinc(full);      // fires when ALL of this lane's copies so far have landed
            __syncwarp();                              // gk / gv are rewritten for the next tile
        };
        // Complete a tile of cnt keys whose per-key meta has been written: zero the rows between
        // the last real one and the end of its 16-key slice (rows past that slice are never
        // looked at: a masked weight is zero, but zero times whatever bits the stage held before
        // need not be), say how full the tile is, and release the plain stores of the whole warp.
        auto pad_tile = [&](int st, int cnt, bool last) {
            uint8_t* k_tile = ring + (size_t)st * L::STAGE_BYTES;
            uint8_t* v_tile = k_tile + L::TILE_BYTES;
            // (the fused small form gives a whole response tile to one warp, which looks at all of it)
            constexpr bool kWholeResp = FUSED && CW == 2 && D <= 128 && NT == 1;
            const int fill = kWholeResp ? TILE : min(TILE, (cnt + 15) & ~15);
            const int zchunks = (fill - cnt) * 8;      // in every 128-byte box the run is contiguous
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx) {
                uint4* kz = reinterpret_cast<uint4*>(k_tile + (size_t)bx * L::BOX_BYTES + (size_t)cnt * 128);
                uint4* vz = reinterpret_cast<uint4*>(v_tile + (size_t)bx * L::BOX_BYTES + (size_t)cnt * 128);
                for (int i = lane; i < zchunks; i += 32) {
                    kz[i] = make_uint4(0u, 0u, 0u, 0u);
                    vz[i] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            if (lane == 0) tile_hdr[st] = make_int2(cnt, last ? 1 : 0);
        };
        auto release_tile = [&](int st) {
            __syncwarp();
            if (lane == 0 && !p.dbg_skip) mbar_arrive(full0 + 8 * st);
        };
        auto finish_tile = [&](int st, int cnt, bool last) {
            pad_tile(st, cnt, last);
            release_tile(st);
        };
        auto publish_tile = [&](int st, int cnt, bool last) {
            copy_rows(st, 0, cnt, true);
            finish_tile(st, cnt, last);
        };
        bool ok = true;
        if constexpr (!FUSED) {
            // ---- rows from the request's list of distinct rows (made by the append kernel) ----
            // A split's range starts at split * quota whatever the row count turns out to be, so
            // the first tile's list entries are requested together with the count, not after it.
            uint2 ucur[UK], unext[UK];          // {row, beam mask} of this lane's keys (lane, lane + 32)
            const int cap = p.W * p.max_steps;
#pragma unroll
            for (int kk = 0; kk < UK; ++kk) {
                const int key = lane + 32 * kk;
                unext[kk] = (p.steps > 0 && key < TILE)
                                ? *reinterpret_cast<const uint2*>(ulist_b + min(split * quota + key, cap - 1))
                                : make_uint2(0u, 0u);
            }
            const int n_b = p.steps > 0 ? p.ucount[b] : 0;
            const int e0 = min(split * quota, n_b);
            const int e1 = (split == SS - 1) ? n_b : min((split + 1) * quota, n_b);
            const int nrt = (e1 - e0 + TILE - 1) / TILE;
            SEGKV_STAMP(4);
            // Tiles [r, r_end) of this CTA's range of the list: row pointers and per-key records into
            // the stage, then the copies.
            int r = 0;
            bool handed = false;
            auto tiles = [&](int r_end) {
                for (; r < r_end && ok; ++r) {
                    const bool own = p.resv && r == 0;            // the stage set aside: nobody else uses it
                    if (!own && !handed) {
                        ok = mbar_wait(hand, 0, p.wait_ns);
                        ok = __all_sync(0xffffffffu, ok);
                        handed = true;
                        if (!ok) break;
                    }
                    const int k = npt + r - p.resv;               // place in the ring's order
                    const int eb = e0 + r * TILE;
                    const int cnt = min(TILE, e1 - eb);
#pragma unroll
                    for (int kk = 0; kk < UK; ++kk) {
                        ucur[kk] = unext[kk];
                        const int key = lane + 32 * kk;
                        unext[kk] = (key < TILE && eb + TILE + key < e1)
                                        ? *reinterpret_cast<const uint2*>(ulist_b + eb + TILE + key)
                                        : make_uint2(0u, 0u);
                    }
                    const int st = own ? rstage : k % RS;
                    if (!own) {
                        ok = mbar_wait(empty0 + 8 * st, (((uint32_t)(k / RS)) & 1) ^ 1, p.wait_ns);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                    }
                    URow* meta_st = meta + (size_t)st * TILE;
#pragma unroll
                    for (int kk = 0; kk < UK; ++kk) {
                        const int key = lane + 32 * kk;
                        if (key >= TILE) continue;
                        const bool valid = key < cnt;
                        const int row = valid ? (int)ucur[kk].x : 0;         // step * rows + slot
                        URow u;
                        u.row = row / p.rows;                                // consumers need the step only
                        u.mask = valid ? ucur[kk].y : 0u;
                        meta_st[key] = u;
                        const int sidx = u.row;
                        gk[key] = k_slab(sidx) + ((size_t)(row - sidx * p.rows) * p.Hkv + kvh) * (size_t)(D * 2);
                    }
                    publish_tile(st, cnt, r == nrt - 1);
                }
            };
            if (gather_ahead) {
                // Lists and rows were written by launches older than this launch's predecessor: the tiles
                // that find a free stage are fetched now, the rows of the others are asked into the L2,
                // and only then does this warp wait for the previous kernel.
                const int r_now = min(nrt, p.resv + (npt < RS ? RS - npt : 0));
                for (int e = e0 + r_now * TILE + lane / 4; e < e1 && p.one_wave; e += 8) {
                    const int row = ulist_b[e].row, sidx = row / p.rows;
                    const char* kr = k_slab(sidx) + ((size_t)(row - sidx * p.rows) * p.Hkv + kvh) * (size_t)(D * 2);
                    const char* src = ((lane & 2) ? kr + p.vdelta : kr) + (lane & 1) * (D);     // K or V row, first or second half
                    prefetch_l2(src);
                    if (D == 256) prefetch_l2(src + 128);
                }
                tiles(r_now);
                grid_wait();
            }
            tiles(nrt);
            SEGKV_STAMP(5);
        } else {
            // ---- fused decode step: rows from the beam-index table, derived on the fly ----
            // The new step's column of the table (Section 3.3) is anc_t[j][s] = anc_{t-1}[parent[j]][s]
            // for s < t and anc_t[j][t] = j.  One lane takes one (step, beam) pair; the lanes of a step
            // compare rows to keep each distinct row once with its beam mask, a warp prefix sum packs
            // the steps of a window densely into the tile, and the column is stored for later steps.
            const int Wb = p.W;
            int Wp = 1;
            while (Wp < Wb) Wp <<= 1;                     // lanes per step (a power of two, <= 16)
            const int spw = 32 / Wp;                      // steps per window
            const int ls = lane / Wp, j = lane % Wp;
            const int gbase = lane - j;                   // first lane of this lane's step
            const int t_new = p.steps - 1;                // the step whose rows are still in k_new / v_new
            constexpr int PF = 4;                         // windows whose table entries are fetched at once
            // Every lane fetches the previous table's entry of its OWN slot j; the entry of its
            // parent slot is then one shuffle away, so the table read does not wait for the parent
            // ids: both requests are in flight together.
            auto fetch_windows = [&](int w0, int (&rowb)[PF]) {
#pragma unroll
                for (int u = 0; u < PF; ++u) {
                    const int s = rs0 + (w0 + u) * spw + ls;
                    rowb[u] = 0;
                    if (s < rs1 && j < Wb && s != t_new) rowb[u] = p.anc_prev[(size_t)(b * Wb + j) * p.max_steps + s];
                }
            };
            // Among the lanes of a step (active ones), keep each distinct row once: `first` marks the
            // lowest lane of a row, `mask` the lanes (slots) that share it; `incl` is the warp-wide
            // running count of first lanes, `total` its last value.
            auto dedupe = [&](int row, bool active, bool& first, uint32_t& mask, int& incl, int& total) {
                if (!active) row = -1 - lane;                                     // matches nobody
                first = active;
                mask = 0;
                for (int i = 0; i < Wp; ++i) {
                    const int ri = __shfl_sync(0xffffffffu, row, gbase + i);
                    if (ri == row) {
                        mask |= 1u << i;
                        if (i < j) first = false;
                    }
                }
                incl = first ? 1 : 0;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += n;
                }
                total = __shfl_sync(0xffffffffu, incl, 31);
            };
            const int nwin = (rs1 - rs0 + spw - 1) / spw;
            const bool has_new = t_new >= rs0 && t_new < rs1;     // this CTA's range holds the step being added
            int rowb[PF];
            // Fast path state: every row this CTA can need, placed in the stage that is its own.
            bool fast = false;
            int fpos[PF];                 // place in the tile of this lane's row (first lane of an old row), or -1
            uint32_t fmask[PF];           // OLD slots whose path holds that row
            int old_total = 0;
            if (gather_ahead) {
                // The previous table and the rows of earlier steps were written by launches older than
                // this launch's predecessor.  The table entries are read now; the rows that any slot's
                // OLD path reaches are a superset of what the new parents will select (the new path of
                // slot j is the old path of slot parent[j]), so they are fetched now, each distinct row
                // once with the set of OLD slots that hold it, and after the wait only the parent ids
                // are a fresh round trip: they turn the old slot sets into the new beams' masks.
                fetch_windows(0, rowb);
                fast = p.resv && nwin <= PF && rs1 > rs0;
                if (fast) {
#pragma unroll
                    for (int u = 0; u < PF; ++u) {
                        fpos[u] = -1;
                        fmask[u] = 0;
                        if (u < nwin) {                                           // warp-uniform
                            const int s = rs0 + u * spw + ls;
                            bool first;
                            int incl, total;
                            dedupe(rowb[u], s < rs1 && j < Wb && s != t_new, first, fmask[u], incl, total);
                            if (first) fpos[u] = old_total + incl - 1;
                            old_total += total;
                        }
                    }
                    if (old_total + (has_new ? Wb : 0) > TILE) fast = false;      // more than the one tile: the general way
                }
                if (fast) {
#pragma unroll
                    for (int u = 0; u < PF; ++u) {
                        if (fpos[u] >= 0) {
                            const int s = rs0 + u * spw + ls;
                            meta[(size_t)rstage * TILE + fpos[u]].row = s;
                            const char* ksl = k_slab(s);
                            const size_t off = ((size_t)rowb[u] * p.Hkv + kvh) * (size_t)(D * 2);
                            gk[fpos[u]] = ksl + off;
                            gv[fpos[u]] = ksl + p.vdelta + off;
                        }
                    }
                    copy_rows(rstage, 0, old_total, false);
                    // where the new step's rows go, their records and the tile's padding are known too
                    if (has_new && lane < Wb) {
                        URow uu;
                        uu.row = t_new;
                        uu.mask = 1u << lane;
                        meta[(size_t)rstage * TILE + old_total + lane] = uu;
                    }
                    pad_tile(rstage, old_total + (has_new ? Wb : 0), true);
                } else if (p.one_wave) {
                    // at least ask the L2 for the rows of the first windows
#pragma unroll
                    for (int u = 0; u < PF; ++u) {
                        const int s = rs0 + u * spw + ls;
                        if (s < rs1 && j < Wb && s != t_new) {
                            const char* kr = k_slab(s) + ((size_t)rowb[u] * p.Hkv + kvh) * (size_t)(D * 2);
#pragma unroll
                            for (int ln = 0; ln < D * 2 / 128; ++ln) {
                                prefetch_l2(kr + ln * 128);
                                prefetch_l2(kr + p.vdelta + ln * 128);
                            }
                        }
                    }
                }
                grid_wait();
                if (fast) {
                    // The new step's rows need nothing but the wait: their copies go out first, straight
                    // from the caller's arrays (CPR lanes per row), and land while the parent ids travel.
                    if (has_new) {
                        const uint32_t k_dst = smem_u32(ring + (size_t)rstage * L::STAGE_BYTES), v_dst = k_dst + L::TILE_BYTES;
                        const int c = lane % CPR;
                        const uint32_t c_off = (uint32_t)(c / 8) * L::BOX_BYTES;
                        for (int r = lane / CPR; r < Wb; r += RPI) {
                            const int key = old_total + r;
                            const uint32_t off = c_off + (uint32_t)key * 128 + (uint32_t)(((c & 7) ^ (key & 7)) << 4);
                            const size_t src = ((size_t)(b * Wb + r) * p.Hkv + kvh) * (size_t)(D * 2) + (size_t)c * 16;
                            cp_async_16(k_dst + off, p.k_new + src);
                            cp_async_16(v_dst + off, p.v_new + src);
                        }
                    }
                    cp_async_mbar_arrive_noinc(full0 + 8 * rstage);      // fires when ALL of this lane's copies, old rows and new, have landed
                }
            }
            int par = j;
            par = (p.steps > 1 && j < Wb) ? p.parent[b * Wb + j] : j;
            if (!gather_ahead) fetch_windows(0, rowb);
            if (j < Wb && (par < 0 || par >= Wb)) {       // first use of the parent ids
                if (kvh == 0 && split == 0) atomicOr(p.err_word, SEGKV_DEV_BAD_PARENT);
                par = par < 0 ? 0 : Wb - 1;
            }
            SEGKV_STAMP(4);
            if (fast) {
                // ---- the rows are on their way: the beam masks, then the new table column ----
                // new slot i reads what old slot parent[i] read: turn the sets of old slots into beam masks
                uint32_t nmask[PF];
#pragma unroll
                for (int u = 0; u < PF; ++u) nmask[u] = 0;
                for (int i = 0; i < Wb; ++i) {
                    const int pi = __shfl_sync(0xffffffffu, par, i);              // lanes 0..Wb-1 hold the slots' parents
#pragma unroll
                    for (int u = 0; u < PF; ++u) nmask[u] |= ((fmask[u] >> pi) & 1u) << i;
                }
#pragma unroll
                for (int u = 0; u < PF; ++u)
                    if (fpos[u] >= 0) meta[(size_t)rstage * TILE + fpos[u]].mask = nmask[u];
                release_tile(rstage);
                // off the consumers' path: the table of the new step
#pragma unroll
                for (int u = 0; u < PF; ++u) {
                    if (u < nwin) {                                               // warp-uniform
                        const int s = rs0 + u * spw + ls;
                        const int row = __shfl_sync(0xffffffffu, rowb[u], gbase + par);   // anc_{t-1}[parent[j]][s]
                        if (s < rs1 && j < Wb && s != t_new && kvh == 0) p.anc_dst[(size_t)(b * Wb + j) * p.max_steps + s] = row;
                    }
                }
                if (has_new && lane < Wb && kvh == 0) p.anc_dst[(size_t)(b * Wb + lane) * p.max_steps + t_new] = b * Wb + lane;
            }
            // Windows of spw steps at fixed positions; the table entries of four windows are
            // requested at once, so a split of up to 4 * spw steps pays one memory round trip.
            // A window (at most 32 rows) is never cut: if it does not fit, the tile is published
            // first and the window opens the next one.
            int fillpos = 0, tix = 0, st = 0;
            bool open = false, handed = false;
            // the tix-th response tile of this CTA: the stage set aside for the first, else the ring
            auto open_tile = [&]() {
                if (p.resv && tix == 0) {
                    st = rstage;
                    open = true;
                    return;
                }
                if (!handed) {
                    ok = mbar_wait(hand, 0, p.wait_ns);
                    ok = __all_sync(0xffffffffu, ok);
                    handed = true;
                    if (!ok) return;
                }
                const int k = npt + tix - p.resv;
                st = k % RS;
                ok = mbar_wait(empty0 + 8 * st, (((uint32_t)(k / RS)) & 1) ^ 1, p.wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                open = ok;
            };
            for (int w0 = 0; w0 < nwin && ok && !fast; w0 += PF) {
                if (w0 > 0) fetch_windows(w0, rowb);
#pragma unroll
                for (int u = 0; u < PF; ++u) {
                    if (w0 + u >= nwin || !ok) break;             // warp-uniform
                    const int s = rs0 + (w0 + u) * spw + ls;
                    const bool active = s < rs1 && j < Wb;
                    int row = __shfl_sync(0xffffffffu, rowb[u], gbase + par);     // anc_{t-1}[parent[j]][s]
                    if (s == t_new) row = b * Wb + j;
                    bool first;
                    uint32_t mask;
                    int incl, total;
                    dedupe(row, active, first, mask, incl, total);
                    if (open && fillpos + total > TILE) {
                        publish_tile(st, fillpos, false);
                        ++tix;
                        open = false;
                        fillpos = 0;
                    }
                    if (!open) {
                        open_tile();
                        if (!ok) break;
                    }
                    if (active) {
                        if (first) {
                            const int pos = fillpos + incl - 1;
                            URow uu;
                            uu.row = s;
                            uu.mask = mask;
                            meta[(size_t)st * TILE + pos] = uu;
                            const size_t off = ((size_t)row * p.Hkv + kvh) * (size_t)(D * 2);
                            const char* ksl = (s == t_new) ? p.k_new : k_slab(s);
                            gk[pos] = ksl + off;
                            gv[pos] = (s == t_new ? p.v_new : ksl + p.vdelta) + off;
                        }
                        if (kvh == 0) p.anc_dst[(size_t)(b * Wb + j) * p.max_steps + s] = row;
                    }
                    fillpos += total;
                }
            }
            if (ok && open) publish_tile(st, fillpos, true);
            SEGKV_STAMP(5);
            // store what the step appends: the parent ids and the new K/V rows of this work group
            if (kvh == 0 && split == 0 && lane < Wb)
                p.parent_row[b * Wb + lane] = p.steps > 1 ? p.parent[b * Wb + lane] : lane;
            if (split == SS - 1) {
                for (int i = lane; i < Wb * CPR; i += 32) {
                    const size_t off = ((size_t)(b * Wb + i / CPR) * p.Hkv + kvh) * (size_t)(D * 2) + (size_t)(i % CPR) * 16;
                    *reinterpret_cast<uint4*>(p.kr_new_slab + off) = *reinterpret_cast<const uint4*>(p.k_new + off);
                    *reinterpret_cast<uint4*>(p.vr_new_slab + off) = *reinterpret_cast<const uint4*>(p.v_new + off);
                }
            }
        }
        if (!ok && lane == 0) {
            atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            s_abort = 1;
        }
    } else {
        // ================================ consumer warps ===============================
        uint32_t qf[NT][KS][2];
        float slope2[NT][2];
        int n_b = 0;
        // accumulators empty; with_inputs: the query fragments, slopes and (separate form) the request's
        // row count, which stays in flight while the prompt tiles are consumed
        auto begin = [&](bool with_inputs) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                m_run[nt][0] = m_run[nt][1] = -INFINITY;
                l_run[nt][0] = l_run[nt][1] = 0.f;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) o_acc[nt][mt][i] = 0.f;
            }
            n_b = (with_inputs && p.steps > 0 && !FUSED) ? p.ucount[b] : 0;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const T* qrow = with_inputs ? qrow_c[nt] : nullptr;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int d0 = ks * 16 + (lane & 3) * 2;
                    qf[nt][ks][0] = qrow ? *reinterpret_cast<const uint32_t*>(qrow + d0) : 0u;
                    qf[nt][ks][1] = qrow ? *reinterpret_cast<const uint32_t*>(qrow + d0 + 8) : 0u;
                }
#pragma unroll
                for (int c = 0; c < 2; ++c)
                    slope2[nt][c] = (with_inputs && slope_c[nt][c]) ? *slope_c[nt][c] * 1.4426950408889634f : 0.f;
            }
        };
        begin(!cons_ahead);
        const int qpos = P + (p.steps > 0 ? p.steps - 1 : -1);

        // One tile: `nvalid` keys exist; for a response tile the per-key beam masks and row
        // ids are in the stage's meta array, for a prompt tile key i sits at position pos0 + i.
        // shared-memory address of 16-byte chunk `ch` of row `key` of a tile (the TMA layout:
        // 128-byte boxes, XOR swizzle; the gather warp writes response rows the same way)
        auto chunk_addr = [&](uint32_t base, int key, int ch, bool) -> uint32_t {
            return base + (uint32_t)(ch >> 3) * L::BOX_BYTES + (uint32_t)key * 128 + (uint32_t)(((ch & 7) ^ (key & 7)) << 4);
        };
        // NB blocks of 16 keys of one tile, at tile-local keys kb0, kb0 + 16, ...: their scores, ONE
        // online-softmax update over all of them, their weighted values.  The blocks are independent
        // until the column maxima meet, so a warp that takes several hides the latency of one
        // block's MMA chain and shuffles behind the others'.
        auto consume = [&](auto nb_c, int st, bool resp, int nvalid, int pos0, int kb0) {
            constexpr int NB = decltype(nb_c)::value;
            if (kb0 >= nvalid) return;
            const uint32_t k_src = smem_u32(ring + (size_t)st * L::STAGE_BYTES);
            const uint32_t v_src = k_src + L::TILE_BYTES;
            // ---- S^T = K . Q^T ----
            float sc[NB][NT][4];
#pragma unroll
            for (int i = 0; i < NB; ++i)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) sc[i][nt][0] = sc[i][nt][1] = sc[i][nt][2] = sc[i][nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const int ch = 2 * ks + (lane >> 4);
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    uint32_t a[4];
                    ldmatrix_x4(a, chunk_addr(k_src, kb0 + 16 * i + (lane & 15), ch, resp));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) Mma<T>::run(sc[i][nt], a, qf[nt][ks][0], qf[nt][ks][1]);
                }
            }
            if (warp == 0 && !resp && pos0 == pt0 * TILE) SEGKV_STAMP(15);
            // ---- mask, bias, online softmax ----
            uint32_t kmask[NB][2];
            float kpos[NB][2];
#pragma unroll
            for (int i = 0; i < NB; ++i)
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int key = kb0 + 16 * i + (lane >> 2) + 8 * r;
                    if (resp) {
                        const URow u = meta[(size_t)st * TILE + key];       // {step, beams that read the row}
                        kmask[i][r] = key < nvalid ? u.mask : 0u;
                        kpos[i][r] = (float)(P + u.row - qpos);
                    } else {
                        kmask[i][r] = key < nvalid ? 0xffffffffu : 0u;
                        kpos[i][r] = (float)(pos0 + key - qpos);
                    }
                }
            // P^T fragments.  bf16 keeps 8 significant bits of a weight, which is not enough where a few
            // keys carry a column's whole weight (a steep ALiBi slope) and their values cancel, so bf16
            // weights go to the tensor cores in two parts, p = hi + lo (16 bits together): the kernel
            // is bound by HBM and the second set of MMAs is free.  fp16 weights (11 bits) go as they are.
            constexpr bool kTwoPart = sizeof(T) == 2 && !Mma<T>::kWeights11Bits;
            uint32_t pfrag[NB][NT][2], pfrag_lo[NB][NT][2];
            bool rescale = false;
            float alpha[NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float s[NB][2][2];
#pragma unroll
                for (int i = 0; i < NB; ++i)
#pragma unroll
                    for (int r = 0; r < 2; ++r)
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            float v = sc[i][nt][2 * r + c] * p.scale2 + slope2[nt][c] * kpos[i][r];
                            s[i][r][c] = (kmask[i][r] & beambit[nt][c]) ? v : -INFINITY;
                        }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float tm = fmaxf(s[0][0][c], s[0][1][c]);
#pragma unroll
                    for (int i = 1; i < NB; ++i) tm = fmaxf(tm, fmaxf(s[i][0][c], s[i][1][c]));
                    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 4));
                    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 8));
                    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 16));
                    const float m_old = m_run[nt][c];
                    const float m_new = fmaxf(m_old, tm);
                    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                    const float a = exp2f(m_old - m_use);
                    alpha[nt][c] = a;
                    rescale = rescale || (a != 1.f);
                    m_run[nt][c] = m_new;
                    float psum = 0.f;
#pragma unroll
                    for (int i = 0; i < NB; ++i) {
                        const float p0 = exp2f(s[i][0][c] - m_use), p1 = exp2f(s[i][1][c] - m_use);
                        s[i][0][c] = p0;
                        s[i][1][c] = p1;
                        psum += p0 + p1;
                    }
                    l_run[nt][c] = l_run[nt][c] * a + psum;
                }
                // P^T as the B operand of O^T += V^T . P^T
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    const uint32_t h0 = Mma<T>::pack(s[i][0][0], s[i][0][1]), h1 = Mma<T>::pack(s[i][1][0], s[i][1][1]);
                    pfrag[i][nt][0] = movmatrix_trans(h0);
                    pfrag[i][nt][1] = movmatrix_trans(h1);
                    if constexpr (kTwoPart) {
                        pfrag_lo[i][nt][0] = movmatrix_trans(Mma<T>::pack(s[i][0][0] - __uint_as_float(h0 << 16), s[i][0][1] - __uint_as_float(h0 & 0xFFFF0000u)));
                        pfrag_lo[i][nt][1] = movmatrix_trans(Mma<T>::pack(s[i][1][0] - __uint_as_float(h1 << 16), s[i][1][1] - __uint_as_float(h1 & 0xFFFF0000u)));
                    }
                }
            }
            if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        o_acc[nt][mt][0] *= alpha[nt][0];
                        o_acc[nt][mt][1] *= alpha[nt][1];
                        o_acc[nt][mt][2] *= alpha[nt][0];
                        o_acc[nt][mt][3] *= alpha[nt][1];
                    }
            }
            // ---- O^T += V^T . P^T ----
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                const int ch = 2 * mt + ((lane >> 3) & 1);
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, chunk_addr(v_src, kb0 + 16 * i + (lane & 7) + 8 * (lane >> 4), ch, resp));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        Mma<T>::run(o_acc[nt][mt], a, pfrag[i][nt][0], pfrag[i][nt][1]);
                        if constexpr (kTwoPart) Mma<T>::run(o_acc[nt][mt], a, pfrag_lo[i][nt][0], pfrag_lo[i][nt][1]);
                    }
                }
            }
        };
        // Small-CTA form: a prompt tile is taken WHOLE by one consumer warp (the warps take turns),
        // its CW blocks side by side; elsewhere every warp takes its own 16 keys of every tile.
        constexpr bool kWholeTile = CW == 2 && D <= 128 && NT == 1;

        bool ok = true;
        int k = 0;
        int st = 0;              // stage and phase of the ring's next tile
        uint32_t ph = 0;
        auto next_stage = [&]() {
            if (++st == RS) {
                st = 0;
                ph ^= 1u;
            }
        };
        if (warp == 0) SEGKV_STAMP(1);
        // k = -1 is the warm-up: the same instructions on whatever the first stage holds, no barrier
        // touched, result thrown away, and then the wait
        if (cons_ahead) k = -1;
        auto warmed_up = [&]() {
            grid_wait();
            if (warp == 0) SEGKV_STAMP(2);
            begin(true);
        };
        // Fused step: one response tile; how many there are and how full each is only the gather warp
        // knows, which says so in the tile's header.  The first has a stage of its own when p.resv.
        int r_done = 0;
        bool resp_last = !(FUSED && rs1 > rs0);
        auto resp_tile = [&]() {
            const bool own = p.resv && r_done == 0;
            const int sr = own ? rstage : st;
            ok = mbar_wait(full0 + 8 * sr, own ? 0u : ph, p.wait_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) return;
            const int2 hd = tile_hdr[sr];
            consume(IntC<1>{}, sr, true, hd.x, 0, warp * 16);
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * sr);
            if (!own) next_stage();
            ++r_done;
            resp_last = hd.y != 0;
        };
        if constexpr (kWholeTile) {
            for (; k < npt; ++k) {
                if constexpr (FUSED) {
                    // The rows of that stage were asked for before the wait, so the tile is there long
                    // before the prompt tiles that had to wait for a stage of the ring: it is consumed
                    // after the first round of prompt tiles, while those reloads travel.
                    if (p.resv && k == RS && !resp_last && r_done == 0) {
                        resp_tile();
                        if (!ok) break;
                    }
                }
                // Every warp waits for every tile, also those it leaves to the other warp, and the stage
                // is released by BOTH: the owner when it has consumed the tile, the other warp as soon as it
                // has seen the tile land.  A parity wait cannot tell a barrier's phases two apart, so a
                // stage must not be refilled (and land) before every warp has seen its current tile:
                // with the owner alone releasing, a warp that fell a tile behind would wait at this
                // barrier for a fill that comes only after a tile it has yet to consume itself.
                if (k >= 0) {
                    ok = mbar_wait(full0 + 8 * st, ph, p.wait_ns);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                if (k < 0 || (k & (CW - 1)) == warp) {
                    const int pos0 = (pt0 + max(k, 0)) * TILE;
                    if (warp == 0 && k == 0) SEGKV_STAMP(7);
                    consume(IntC<CW>{}, k < 0 ? 0 : st, false, min(TILE, P - pos0), pos0, 0);
                    if (warp == 0 && k == 0) SEGKV_STAMP(6);
                    __syncwarp();
                    if (k >= 0 && lane == 0) mbar_arrive(empty0 + 8 * st);
                } else if (lane == 0) {
                    mbar_arrive(empty0 + 8 * st);
                }
                if (k < 0) warmed_up();
                else next_stage();
            }
        }
        for (; k < npt; ++k) {
            if (k >= 0) {
                ok = mbar_wait(full0 + 8 * st, ph, p.wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
            }
            const int pos0 = (pt0 + max(k, 0)) * TILE;
            if (warp == 0 && k == 0) SEGKV_STAMP(7);
            consume(IntC<1>{}, k < 0 ? 0 : st, false, min(TILE, P - pos0), pos0, warp * 16);
            if (warp == 0 && k == 0) SEGKV_STAMP(6);
            __syncwarp();
            if (k < 0) warmed_up();
            else {
                if (lane == 0) mbar_arrive(empty0 + 8 * st);
                next_stage();
            }
        }
        if (warp == 0) SEGKV_STAMP(8);
        if (ok && !FUSED) {
            const int e0 = min(split * quota, n_b);
            const int e1 = (split == SS - 1) ? n_b : min((split + 1) * quota, n_b);
            const int nrt = (e1 - e0 + TILE - 1) / TILE;
            for (int r = 0; r < nrt; ++r, ++k) {
                const bool own = p.resv && r == 0;                // the first response tile has a stage of its own
                const int sr = own ? rstage : st;
                ok = mbar_wait(full0 + 8 * sr, own ? 0u : ph, p.wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                consume(IntC<1>{}, sr, true, min(TILE, e1 - (e0 + r * TILE)), 0, warp * 16);
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * sr);
                if (!own) next_stage();
            }
        } else {
            while (ok && !resp_last) resp_tile();
        }
        if (!ok && lane == 0) {
            atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            s_abort = 1;
        }
        cons_ok = ok;
    }

    if (warp == 0) SEGKV_STAMP(9);
    // ==================================== epilogue ====================================
    if (p.cluster) {
        // ---- split merge inside the thread-block cluster, through distributed shared memory ----
        // Only the consumer warps take part, and nobody meets at a cluster barrier: the (column, d)
        // plane is cut into S equal slices, CTA r merges slice r, every CTA sends its part of
        // slice r to CTA r with stores that report their bytes to CTA r's receive barrier, and CTA r
        // folds the S partials once its own barrier says they are all there.
        constexpr int CT = CW * 32;                       // consumer threads
        const int ncols = p.ncols, S = p.S;
        const int slice = ncols * D / S;                  // floats; a multiple of 4
        if (warp < CW) {
            float* mrg_o = reinterpret_cast<float*>(smem);                       // [CW][8*NT][DP], over the ring
            float* mrg_ml = mrg_o + (size_t)CW * 8 * NT * DP;                    // [CW][8*NT][2]
            named_bar_sync(1, CT);                        // every consumer warp is done reading the ring
            const bool bad = !cons_ok || *reinterpret_cast<volatile int*>(&s_abort) != 0;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float l = l_run[nt][c];
                    l += __shfl_xor_sync(0xffffffffu, l, 4);
                    l += __shfl_xor_sync(0xffffffffu, l, 8);
                    l += __shfl_xor_sync(0xffffffffu, l, 16);
                    const int col = nt * 8 + (lane & 3) * 2 + c;
                    if ((lane >> 2) == 0) {
                        mrg_ml[((size_t)warp * 8 * NT + col) * 2 + 0] = m_run[nt][c];
                        mrg_ml[((size_t)warp * 8 * NT + col) * 2 + 1] = l;
                    }
                    float* dst = mrg_o + ((size_t)warp * 8 * NT + col) * DP + (lane >> 2);
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        dst[mt * 16] = o_acc[nt][mt][c];
                        dst[mt * 16 + 8] = o_acc[nt][mt][2 + c];
                    }
                }
            }
            named_bar_sync(1, CT);
            if (tid == 0) SEGKV_STAMP(10);
            const uint32_t me = cluster_ctarank();
            const float inv_slice4 = 4.f / (float)slice;
            cluster_wait_acquire();                       // every CTA of the cluster has set its barrier up
            for (int it = tid; it < ncols * D4; it += CT) {
                const int col = it / D4, d = (it % D4) * 4;
                // merged partial of this CTA for one float4 of one column
                float mm = -INFINITY;
#pragma unroll
                for (int w = 0; w < CW; ++w) mm = fmaxf(mm, mrg_ml[((size_t)w * 8 * NT + col) * 2]);
                float ll = 0.f;
                float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < CW; ++w) {
                    const float mw = mrg_ml[((size_t)w * 8 * NT + col) * 2];
                    const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - mm);
                    ll += mrg_ml[((size_t)w * 8 * NT + col) * 2 + 1] * f;
                    const float4 v = *reinterpret_cast<const float4*>(mrg_o + ((size_t)w * 8 * NT + col) * DP + d);
                    o.x += v.x * f; o.y += v.y * f; o.z += v.z * f; o.w += v.w * f;
                }
                const int f4 = col * D4 + (d >> 2);                              // float4 index in the plane
                const int r = (int)(((float)f4 + 0.5f) * inv_slice4);            // its slice (exact: small integers)
                const uint32_t rbar = mapa_shared(recvbar, (uint32_t)r);
                st_async_v4(mapa_shared(smem_u32(recv_o + (size_t)me * slice + 4 * f4 - r * slice), (uint32_t)r), o, rbar);
                if (d == 0) {
                    // a CTA that gave up says so with a NaN sum (and no weight): the sum of the fold is then NaN
                    // and its peers leave the output alone
                    if (bad) {
                        mm = -INFINITY;
                        ll = __int_as_float(0x7fc00000);
                    }
                    for (int r2 = 0; r2 < S; ++r2)
                        st_async_v2(mapa_shared(smem_u32(recv_ml + ((size_t)me * ncols + col) * 2), (uint32_t)r2), mm, ll,
                                    mapa_shared(recvbar, (uint32_t)r2));
                }
            }
            if (tid == 0) SEGKV_STAMP(14);
            bool got = mbar_wait_cluster(recvbar, 0, p.wait_ns);
            got = __all_sync(0xffffffffu, got);
            if (tid == 0) SEGKV_STAMP(12);
            if (!got && lane == 0) atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            // fold: one thread per float of the slice; the S partials of that float and their {max, sum}
            // pairs are all asked for at once, no lane talks to another
            for (int e = tid; e < slice && got; e += CT) {
                const int fl = (int)me * slice + e;
                const int col = fl / D, d = fl % D;
                float mp[kMaxCluster], lp[kMaxCluster], vp[kMaxCluster];
#pragma unroll
                for (int sp = 0; sp < kMaxCluster; ++sp) {
                    const bool in = sp < S;
                    const float2 ml = in ? *reinterpret_cast<const float2*>(recv_ml + ((size_t)sp * ncols + col) * 2)
                                         : make_float2(-INFINITY, 0.f);
                    mp[sp] = ml.x;
                    lp[sp] = ml.y;
                    vp[sp] = in ? recv_o[(size_t)sp * slice + e] : 0.f;
                }
                float mm = mp[0];
#pragma unroll
                for (int sp = 1; sp < kMaxCluster; ++sp) mm = fmaxf(mm, mp[sp]);
                float ll = 0.f, v = 0.f;
#pragma unroll
                for (int sp = 0; sp < kMaxCluster; ++sp) {
                    const float f = (mp[sp] == -INFINITY) ? 0.f : exp2f(mp[sp] - mm);
                    ll += lp[sp] * f;                       // NaN from a CTA that gave up stays NaN
                    v += vp[sp] * f;
                }
                if (ll == ll) {
                    const int j = col / p.G, hg = col % p.G;
                    T* orow = reinterpret_cast<T*>(p.out) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D + d;
                    *orow = Mma<T>::down(v * (1.f / ll));
                }
            }
            if (tid == 0) SEGKV_STAMP(13);
        }
        // the CTA leaves together: a producer warp that gave up first lets its copies in flight land
        __syncthreads();
        if (s_abort != 0) {
            if (warp == TMA_WARP)
                for (int k = max(0, tma_issued - stages); k < tma_issued; ++k)
                    (void)mbar_wait(full0 + 8 * (k % RS), (uint32_t)(k / RS) & 1, p.wait_ns);
            if (warp == GATHER_WARP) cp_async_wait_all();
        }
        return;
    }
    __syncthreads();
    if (tid == 0) SEGKV_STAMP(10);
    const bool aborted = s_abort != 0;
    if (aborted) {
        // Something never arrived.  Give copies still in flight a bounded chance to land
        // before the shared memory is released; the output is left untouched.
        if (warp == TMA_WARP)
            for (int k = max(0, tma_issued - stages); k < tma_issued; ++k)
                (void)mbar_wait(full0 + 8 * (k % RS), (uint32_t)(k / RS) & 1, p.wait_ns);
        if (warp == GATHER_WARP) cp_async_wait_all();
    }

    // ---- merge the consumer warps (each saw a different quarter of every tile) ----
    float* mrg_o = reinterpret_cast<float*>(smem);                       // [CW][8*NT][DP]
    float* mrg_ml = mrg_o + (size_t)CW * 8 * NT * DP;                    // [CW][8*NT][2]
    if (warp < CW && !aborted) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                float l = l_run[nt][c];
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                const int col = nt * 8 + (lane & 3) * 2 + c;
                if ((lane >> 2) == 0) {
                    mrg_ml[((size_t)warp * 8 * NT + col) * 2 + 0] = m_run[nt][c];
                    mrg_ml[((size_t)warp * 8 * NT + col) * 2 + 1] = l;
                }
                float* dst = mrg_o + ((size_t)warp * 8 * NT + col) * DP + (lane >> 2);
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    dst[mt * 16] = o_acc[nt][mt][c];
                    dst[mt * 16 + 8] = o_acc[nt][mt][2 + c];
                }
            }
        }
    }
    __syncthreads();

    const int ncols = p.ncols;
    const int S = SS;
    // merged partial of this CTA for one float4 of one column
    auto merged = [&](int col, int d, float& mm, float& ll) -> float4 {
        mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < CW; ++w) mm = fmaxf(mm, mrg_ml[((size_t)w * 8 * NT + col) * 2]);
        ll = 0.f;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < CW; ++w) {
            const float mw = mrg_ml[((size_t)w * 8 * NT + col) * 2];
            const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - mm);
            ll += mrg_ml[((size_t)w * 8 * NT + col) * 2 + 1] * f;
            const float4 v = *reinterpret_cast<const float4*>(mrg_o + ((size_t)w * 8 * NT + col) * DP + d);
            o.x += v.x * f; o.y += v.y * f; o.z += v.z * f; o.w += v.w * f;
        }
        return o;
    };
    auto store_out = [&](int col, int d, float4 o) {
        const int j = col / p.G, hg = col % p.G;
        T* orow = reinterpret_cast<T*>(p.out) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D + d;
        uint2 pk;
        pk.x = Mma<T>::pack(o.x, o.y);
        pk.y = Mma<T>::pack(o.z, o.w);
        *reinterpret_cast<uint2*>(orow) = pk;
    };

    if (aborted) {
        // The work group's arrival counter must still come back to zero for the next launch: take the
        // ticket, marked, so that the last CTA to arrive skips the merge (the output stays untouched).
        if (S > 1 && tid == 0) {
            int ticket;
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(ticket) : "l"(p.tickets + slab), "r"(kTicketAborted + 1) : "memory");
            if ((ticket & (kTicketAborted - 1)) == S - 1) p.tickets[slab] = 0;
        }
        return;
    }

    float* wso_cta = p.ws_o + (size_t)ws_item * ncols * D;
    float* wsml_cta = p.ws_ml + (size_t)ws_item * ncols * 2;
    for (int it = tid; it < ncols * D4; it += NTHREADS) {
        const int col = it / D4, d = (it % D4) * 4;
        float mm, ll;
        float4 o = merged(col, d, mm, ll);
        if (S == 1) {
            const float inv = 1.f / ll;
            o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
            store_out(col, d, o);
        } else {
            *reinterpret_cast<float4*>(wso_cta + (size_t)col * D + d) = o;
            if (d == 0) *reinterpret_cast<float2*>(wsml_cta + col * 2) = make_float2(mm, ll);
        }
    }
    if (tid == 0) SEGKV_STAMP(11);
    if (S == 1) return;

    // ---- split merge through the global workspace: the last CTA of the work group to
    // ---- arrive (atomic ticket, nobody waits) merges all partials
    __syncthreads();
    if (tid == 0) {
        // release: this CTA's partials (ordered before by the barrier) are visible before the
        // ticket; acquire: the last arriver sees every other CTA's partials
        int ticket;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(ticket) : "l"(p.tickets + slab) : "memory");
        s_last = (ticket & (kTicketAborted - 1)) == S - 1 ? 1 + (ticket >= kTicketAborted ? 1 : 0) : 0;
        if (s_last == 2) p.tickets[slab] = 0;     // a CTA of the group gave up: no merge, counter ready for the next launch
    }
    __syncthreads();
    if (tid == 0) SEGKV_STAMP(12);
    if (s_last != 1) return;

    // One pass: each thread owns a float4 of one column and folds the splits in, eight at a
    // time (their partial outputs and max/sum pairs are all requested before any is used).
    const float2* wsml_slab = reinterpret_cast<const float2*>(p.ws_ml + (size_t)(ws_item - split) * ncols * 2);
    const float* wso_slab = p.ws_o + (size_t)(ws_item - split) * ncols * D;
    for (int it = tid; it < ncols * D4; it += NTHREADS) {
        const int col = it / D4, d = (it % D4) * 4;
        const float4* src = reinterpret_cast<const float4*>(wso_slab + (size_t)col * D + d);
        const size_t sstride = (size_t)ncols * D4;            // float4 per split
        float mm = -INFINITY, ll = 0.f;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < S; s0 += 8) {
            float4 v[8];
            float2 ml[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const bool in = s0 + u < S;
                ml[u] = in ? __ldcg(wsml_slab + (size_t)(s0 + u) * ncols + col) : make_float2(-INFINITY, 0.f);
                v[u] = in ? __ldcg(src + (size_t)(s0 + u) * sstride) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float bm = mm;
#pragma unroll
            for (int u = 0; u < 8; ++u) bm = fmaxf(bm, ml[u].x);
            const float fo = (mm == -INFINITY) ? 0.f : exp2f(mm - bm);
            ll *= fo; o.x *= fo; o.y *= fo; o.z *= fo; o.w *= fo;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float f = (ml[u].x == -INFINITY) ? 0.f : exp2f(ml[u].x - bm);
                ll += ml[u].y * f;
                o.x += v[u].x * f; o.y += v[u].y * f; o.z += v[u].z * f; o.w += v[u].w * f;
            }
            mm = bm;
        }
        const float inv = 1.f / ll;
        o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
        store_out(col, d, o);
    }
    if (tid == 0) p.tickets[slab] = 0;      // ready for the next launch
    if (tid == 0) SEGKV_STAMP(13);
}

template <typename T, int D, int NT, int CW, bool FUSED>
cudaError_t launch_one(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv, int stages,
                       cudaStream_t st) {
    using L = Layout<D, CW>;
    const size_t smem = L::bytes(stages, NT);
    auto kern = sdpa_tiled_kernel<T, D, NT, CW, FUSED>;
    static size_t configured[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && configured[dev] < smem) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = smem;
    }
    TiledParams p;
    p.q = a.q; p.out = a.out; p.slopes = a.slopes;
    p.kr = (const char*)a.kr; p.k_chunks = (const char* const*)a.k_chunks; p.vdelta = a.vdelta;
    p.chunk_steps = d.chunk_steps;
    p.ulist = a.ulist; p.ucount = a.ucount; p.tickets = a.tickets; p.err_word = a.err_word;
    p.fused = a.fused ? 1 : 0;
    p.anc_prev = a.anc; p.parent = a.parent; p.k_new = (const char*)a.k_new; p.v_new = (const char*)a.v_new;
    p.kr_new_slab = (char*)a.kr_new_slab; p.vr_new_slab = (char*)a.vr_new_slab;
    p.anc_dst = a.anc_dst; p.parent_row = a.parent_row;
    p.plens = a.plens;
    p.P = a.prompt_len; p.steps = a.steps; p.S = a.splits; p.W = d.beams; p.G = d.group; p.H = d.heads;
    p.Hkv = d.kv_heads; p.rows = d.rows; p.max_steps = d.max_steps; p.ncols = d.beams * d.group; p.stages = stages;
    p.scale2 = 1.4426950408889634f / sqrtf((float)D);
    p.quota = (a.steps + 2 * d.beams + a.splits - 1) / a.splits;
    if (p.quota < 1) p.quota = 1;
    const size_t slabs = (size_t)d.batch * d.kv_heads;
    const int tail_groups = (a.tail_groups > 0 && a.tail_splits > 0 && !a.cluster) ? a.tail_groups : 0;
    p.tail_groups = tail_groups;
    p.tail_S = tail_groups ? a.tail_splits : a.splits;
    p.tail_quota = (a.steps + 2 * d.beams + p.tail_S - 1) / p.tail_S;
    if (p.tail_quota < 1) p.tail_quota = 1;
    p.head_items = (int)((slabs - tail_groups) * a.splits);
    // work groups that are not split store their output directly: the workspace then starts at the tail
    p.ws_item0 = (tail_groups && a.splits == 1) ? p.head_items : 0;
    const size_t items = (size_t)p.head_items + (size_t)tail_groups * p.tail_S;
    p.cluster = a.cluster ? 1 : 0;
    p.early_prompt = (a.pdl && a.prompt_immutable) ? 1 : 0;
    p.early_rows = (a.pdl && a.prompt_immutable && a.rows_immutable) ? 1 : 0;
    p.one_wave = a.one_wave ? 1 : 0;
    p.resv = (p.early_rows && a.one_wave && stages >= 2) ? 1 : 0;
    p.dbg_skip = a.dbg_skip ? 1 : 0;
    p.wait_ns = a.wait_ns ? a.wait_ns : kWaitLimitNs;
#ifdef SEGKV_TIMELINE
    static int launch_id = 0;
    p.dbg_launch = launch_id++;
#endif
    p.ws_o = a.ws;
    p.ws_ml = a.ws ? a.ws + (items - p.ws_item0) * p.ncols * D : nullptr;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)items, 1, 1);
    cfg.blockDim = dim3(32 * (CW + 2), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    unsigned na = 0;
    if (p.cluster) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)a.splits;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (a.pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = na ? attr : nullptr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, tmk, tmv, p);
}

template <typename T>
cudaError_t dispatch(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv, int stages,
                     cudaStream_t st) {
    const int nt = (d.beams * d.group + 7) / 8;
    if (a.splits < 1 || a.splits > kMaxSplits) return cudaErrorInvalidValue;
    if (a.cluster && !tiled_cluster_ok(d, a.splits)) return cudaErrorInvalidValue;
    if (nt == 1 && a.small && d.head_dim <= 128) {
        // 32-key tiles, two consumer warps: a CTA of a quarter of an SM, for launches of at most one wave
        if (d.head_dim == 64) return a.fused ? launch_one<T, 64, 1, 2, true>(d, a, tmk, tmv, stages, st)
                                             : launch_one<T, 64, 1, 2, false>(d, a, tmk, tmv, stages, st);
        return a.fused ? launch_one<T, 128, 1, 2, true>(d, a, tmk, tmv, stages, st)
                       : launch_one<T, 128, 1, 2, false>(d, a, tmk, tmv, stages, st);
    }
    if (nt == 1) {
        switch (d.head_dim) {
            case 64: return a.fused ? launch_one<T, 64, 1, 4, true>(d, a, tmk, tmv, stages, st)
                                    : launch_one<T, 64, 1, 4, false>(d, a, tmk, tmv, stages, st);
            case 128: return a.fused ? launch_one<T, 128, 1, 4, true>(d, a, tmk, tmv, stages, st)
                                    : launch_one<T, 128, 1, 4, false>(d, a, tmk, tmv, stages, st);
            case 256: return a.fused ? launch_one<T, 256, 1, 2, true>(d, a, tmk, tmv, stages, st)
                                    : launch_one<T, 256, 1, 2, false>(d, a, tmk, tmv, stages, st);
        }
    } else if (nt == 2) {
        switch (d.head_dim) {
            case 64: return a.fused ? launch_one<T, 64, 2, 4, true>(d, a, tmk, tmv, stages, st)
                                    : launch_one<T, 64, 2, 4, false>(d, a, tmk, tmv, stages, st);
            case 128: return a.fused ? launch_one<T, 128, 2, 4, true>(d, a, tmk, tmv, stages, st)
                                    : launch_one<T, 128, 2, 4, false>(d, a, tmk, tmv, stages, st);
        }
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool tiled_supported(const Dims& d) {
    const int nt = (d.beams * d.group + 7) / 8;
    return nt == 1 || (nt == 2 && d.head_dim <= 128);
}

// The cluster combine needs a portable cluster size and equal float4-aligned slices.
bool tiled_cluster_ok(const Dims& d, int splits) {
    if (splits != 2 && splits != 4 && splits != 8) return false;
    return ((long long)d.beams * d.group * d.head_dim) % (4LL * splits) == 0;
}

bool tiled_small_ok(const Dims& d) { return d.head_dim <= 128 && d.beams * d.group <= 8; }

int tiled_tile_keys(int head_dim, bool small) { return (head_dim == 256 || small) ? 32 : 64; }

size_t tiled_smem_bytes(const Dims& d, int stages, bool small) {
    const int nt = (d.beams * d.group + 7) / 8;
    if (small && tiled_small_ok(d)) return d.head_dim == 64 ? Layout<64, 2>::bytes(stages, nt) : Layout<128, 2>::bytes(stages, nt);
    switch (d.head_dim) {
        case 64: return Layout<64, 4>::bytes(stages, nt);
        case 128: return Layout<128, 4>::bytes(stages, nt);
        default: return Layout<256, 2>::bytes(stages, nt);
    }
}

cudaError_t launch_sdpa_tiled(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv,
                              int stages, cudaStream_t st) {
    return d.dtype == SEGKV_BF16 ? dispatch<__nv_bfloat16>(d, a, tmk, tmv, stages, st)
                                 : dispatch<__half>(d, a, tmk, tmv, stages, st);
}

}  // namespace segkv_impl

// ---------------------------------------------------------------------------
// Variant of the launcher for callers that must not allocate: the split
// workspace (partial outputs, their max/sum and the arrival tickets of the
// workspace combine) lives in a fixed array that is part of the loaded module.
// ---------------------------------------------------------------------------
namespace segkv_impl {

constexpr size_t kStaticScratchBytes = (size_t)8 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

size_t tiled_static_scratch_bytes() { return kStaticScratchBytes; }

// Returns cudaSuccess with *too_big = 1 (nothing launched) when the launch shape needs
// more scratch than the array holds.
cudaError_t launch_sdpa_tiled_static(const Dims& d, SdpaArgs a, const CUtensorMap& tmk, const CUtensorMap& tmv,
                                     int stages, cudaStream_t st, int* too_big) {
    *too_big = 0;
    // In host code the array's name is only a handle for the runtime, not a device address:
    // ask for the address once per device (with that device current) and keep it.
    static void* base_of[64] = {nullptr};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    void* base = (dev >= 0 && dev < 64) ? base_of[dev] : nullptr;
    if (!base) {
        e = cudaGetSymbolAddress(&base, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) base_of[dev] = base;
    }
    const size_t slabs = (size_t)d.batch * d.kv_heads;
    const size_t ticket_bytes = (slabs * sizeof(int) + 255) & ~(size_t)255;
    const size_t ws_bytes = slabs * a.splits * d.beams * d.group * (d.head_dim + 2) * sizeof(float);
    if (a.splits > 1) {
        if (ticket_bytes + ws_bytes > kStaticScratchBytes) {
            *too_big = 1;
            return cudaSuccess;
        }
        // the tickets must read zero at the start of every launch; the array keeps whatever
        // the last call (of any handle) left there
        e = cudaMemsetAsync(base, 0, ticket_bytes, st);
        if (e != cudaSuccess) return e;
    }
    a.tickets = reinterpret_cast<int*>(base);
    a.ws = reinterpret_cast<float*>(static_cast<unsigned char*>(base) + ticket_bytes);
    a.cluster = false;
    return launch_sdpa_tiled(d, a, tmk, tmv, stages, st);
}

}  // namespace segkv_impl

#ifdef SEGKV_TIMELINE
extern "C" __attribute__((visibility("default"))) int segkv_debug_timeline(unsigned long long* host, int clear) {
    if (cudaMemcpyFromSymbol(host, segkv_impl::g_timeline, sizeof(unsigned long long) * 8 * 512 * 32) != cudaSuccess) return -1;
    if (clear) {
        void* p = nullptr;
        cudaGetSymbolAddress(&p, segkv_impl::g_timeline);
        cudaMemset(p, 0, sizeof(unsigned long long) * 8 * 512 * 32);
    }
    return 0;
}
#endif
