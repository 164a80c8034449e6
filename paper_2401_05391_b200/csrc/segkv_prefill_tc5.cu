// Prefill attention on the fifth-generation tensor cores (tcgen05 + tensor memory), head_dim 64,
// 128 or 256 (paper Section 3.1 / 3.3: the prefill kernel is the special case of the customised
// SDPA kernel that sees only the query and the prompt key/value, batch-first in and out):
//     out[b,i,h,:] = softmax_{j<=i}( q[b,i,h,:] . K[b,j,:] / sqrt(D) + bias ) . V[b,j,:].
//
//   * one persistent CTA per SM walks a static list of work items (one or two groups of 128
//     query rows of one (request, head)), longest first; a group's rows are one per TMEM lane and
//     per softmax thread;
//   * Q of each group arrives by TMA (a per-call tensor map over [B, N, H, D]) in the
//     128-byte-swizzled K-major layout; K and V tiles (128 keys; 64 at head_dim 256) arrive by TMA
//     in the same layout through separate rings: a K tile is needed one step before the V tile
//     of the same keys.  They come from the prompt segment, or (fused prefill) from the caller's
//     arrays, and are then also stored on into the segment, each tile by one CTA;
//   * one elected thread issues the MMAs: S = Q.K^T (M 128, N = keys of a tile, K-steps of 16)
//     into a TMEM buffer and O += P.V (M 128, N = head_dim) into a TMEM accumulator.  P never
//     touches shared memory: the softmax threads write it, rounded to the 16-bit type, over the
//     first half of the columns of the S buffer it came from, and the MMA takes its A operand
//     from tensor memory.  V is consumed as an MN-major B operand straight from its row-major
//     tile;
//   * the softmax threads read S with tcgen05.ld (no shuffles for the row max / sum) and
//     rescale O in tensor memory only when a row's maximum has grown by more than 2^8 since the
//     reference it is using (the sum uses the same reference, so the result is exact);
//   * with two groups per CTA each has one S buffer and the tensor cores work for one group
//     while the other is in its softmax; with one group S is double-buffered so that Q.K^T of
//     tile j+1 runs under the softmax of tile j.  The tail of one item overlaps the head of the
//     next (loads, and the first Q.K^T while the previous output is stored).
//
// Tensor memory (all 512 columns are allocated): S buffers first, then one O accumulator per
// group.  Every mbarrier is waited on phase by phase (a parity wait cannot tell phases two
// apart) and every wait is bounded; on expiry the kernel flags SEGKV_DEV_WAIT_LIMIT, skips
// the output and still releases its tensor memory.
#include "segkv_internal.h"
#include "segkv_ptx.cuh"

namespace segkv_impl {

namespace {

using namespace ptx;

constexpr int kRows = 128;     // query rows per group (TMEM lanes)
constexpr int kBoxQ = kRows * 128;           // 64 head-dim elements of a group's Q rows (one 128-byte swizzle span wide)
constexpr int kTmemCols = 512;

struct Tc5Params {
    const void* q;
    void* out;
    const float* slopes;
    int* err_word;
    const int32_t* plens;    // per-request prompt lengths (rows and keys past them are skipped), or NULL
    int N, H, Hkv, G, B, snake;
    int paired, rounds;      // item order: see round_item; rounds = items a CTA walks through (some may be empty)
    int store_kv;            // 1: every K/V tile is also written to the prompt segment, by the item that owns it
    float scale2;
    uint32_t idesc_qk, idesc_pv;
    int dbg_skip;            // test aid: one softmax thread leaves out one barrier arrival, so that a wait runs out
    unsigned long long wait_ns;   // limit of every bounded wait
};

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] . B[smem]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// D[tmem] (+)= A[tmem] . B[smem]; A is M x 16 of a 16-bit type, two elements per 32-bit column
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// 32 lanes x 32 columns of 32-bit words: this thread's TMEM lane, 32 consecutive columns
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  K-major operands: rows of 128 bytes, eight
// rows (1024 B) per swizzle atom, SBO = distance between atoms of eight rows, LBO unused (1).
// MN-major operands (V: rows are keys = the K dimension, 64 contiguous MN elements per row):
// SBO = distance between groups of eight K rows, LBO = distance between 64-element MN blocks.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
    const uint32_t hi = (sbo_bytes >> 4) | (1u << 14) /* descriptor version */ | (2u << 29) /* SWIZZLE_128B */;
    return ((uint64_t)hi << 32) | lo;
}

template <bool B> struct BoolC { static constexpr bool value = B; };
template <typename T> struct SplitP { typedef char yes; static constexpr bool value = false; };
template <> struct SplitP<__nv_bfloat16> { typedef char yes; static constexpr bool value = true; };

// Critical-path wait: poll without sleeping first (the hardware suspends the thread inside
// try_wait for a while), then fall back to the bounded, sleeping wait.
__device__ __forceinline__ bool mbar_wait_hot(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
#pragma unroll 1
    for (int i = 0; i < 4096; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, limit_ns);
}

#ifdef SEGKV_TC5_TIMELINE
}  // namespace
__device__ long long g_tc5_tl[3 * 64 * 8];
#define TC5_STAMP(role, kt, ev)                                                                   \
    do {                                                                                          \
        if ((SEGKV_TC5_TIMELINE != 2 || ((role) == 2 && (ev) == 0)) &&                            \
            w == 0 && (kt) < 64)                                                                 \
            g_tc5_tl[((role) * 64 + (kt)) * 8 + (ev)] = clock64();                                \
    } while (0)
namespace {
#else
#define TC5_STAMP(role, kt, ev) do {} while (0)
#endif

// Shape of one instantiation: head_dim D (64, 128 or 256), KEYS keys per K/V tile, NG groups of
// 128 query rows per CTA.  head_dim 256 leaves tensor memory for one group and 64-key tiles only.
template <int D_, int KEYS_, int NG_>
struct Tc5Layout {
    static constexpr int D = D_, KEYS = KEYS_, NG = NG_;
    static constexpr int NB = NG == 1 ? 2 : 1;                   // S buffers per group
    static constexpr int kThreads = 32 * (4 * NG + 2);
    static constexpr int kDBoxes = D / 64;                       // 64-element (128-byte) column blocks of a row
    static constexpr int kBoxRows = D == 256 ? 32 : 64;          // rows of one TMA box of the prompt segment's tensor map
    static constexpr int kBoxBytes = kBoxRows * 128;
    static constexpr int kColTile = KEYS * 128;                  // one column block of all keys of a tile
    static constexpr int kTileKV = kDBoxes * kColTile;           // bytes of a K (or a V) tile
    static constexpr int kStagesK = 3;
    static constexpr int kStagesV = (NG == 1 && D <= 128) ? 3 : 2;
    static constexpr int kRingK = kStagesK * kTileKV;
    static constexpr int kRingV = kStagesV * kTileKV;
    static constexpr int kQGroup = kDBoxes * kBoxQ;              // bytes of one group's Q
    static constexpr int kQ = NG * kQGroup;
    static constexpr int kBars = 2 * kStagesK + 2 * kStagesV + 6 * NG;   // K full/empty, V full/empty, per group: S0 S1 P O Qfull Qempty
    static constexpr size_t kBytes = 1024 + (size_t)kRingK + kRingV + kQ + 8 * kBars + 64;
    // tensor memory: S buffers of KEYS columns first, then one O accumulator of D columns per group
    static constexpr int kColO = NG * NB * KEYS;
    static_assert(kColO + NG * D <= kTmemCols, "tensor memory");
    static_assert(kBytes <= 232448, "shared memory");
};

// Row maximum of one tile's scores.  BIAS: sv[i] <- sv[i] * scale2 + slope2 * (key_i - row), the
// maximum is in log2 units; otherwise sv keeps the raw dot products and the maximum is raw.
// MASK: keys above the row (i > lim) are set to -inf first.
template <int KEYS, bool BIAS, bool MASK>
__device__ __forceinline__ float score_max(float* sv, float scale2, float slope2, float bias0, int lim) {
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < KEYS; ++i) {
        float v = sv[i];
        if (BIAS) v = fmaf(v, scale2, fmaf(slope2, (float)i, bias0));
        if (MASK) v = i > lim ? -INFINITY : v;
        if (BIAS || MASK) sv[i] = v;
        mx[i & 3] = fmaxf(mx[i & 3], v);
    }
    return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
}

// bf16 keeps 8 significant bits of a softmax weight.  Where a few keys carry a row's whole weight
// and their values cancel, that rounding alone exceeds the path's tolerance, so where it can
// happen the weights go to the tensor cores as TWO bf16 parts, p = hi + lo (hi = p cut to bf16,
// lo = bf16(p - hi): 16 significant bits together), lo in the second half of the S buffer's
// columns, and O takes a second P.V MMA for those keys.  Which keys is known from the launch
// shape: the first key tile of the rows that start the prompt (a handful of keys in all), and,
// under an ALiBi slope steep enough to put a row's weight on its nearest neighbours, the keys
// within kSplitWindow of the group's rows.  fp16 weights (11 bits) never need it.
constexpr float kSplitSlope = 0.0625f;   // weights fall by e^-slope per key: below this, dozens of keys share a row's weight
constexpr int kSplitWindow = 64;
// Do the `nkeys` keys from `key0` on get two-part weights, for the group whose first row is row0?
__device__ __forceinline__ bool split_p_keys(int row0, int key0, int nkeys, float slope) {
    if (row0 == 0 && key0 < kRows) return true;
    return slope >= kSplitSlope && key0 + nkeys - 1 >= row0 - kSplitWindow;
}

// One CTA per SM walks a static list of work items (128*NG query rows of one (request, head)),
// longest first and dealt round-robin, so that the tail of one item overlaps the head of the
// next: the producer runs ahead through the K/V rings and reloads a group's Q as soon as the
// group's last Q.K^T has been read, and the first Q.K^T of the next item executes while the
// softmax threads are still storing the previous output.
// MODE 0: K/V from the prompt segment, one prompt length; 1: fused prefill (K/V from the caller's arrays,
// every tile stored into the segment); 2: per-request prompt lengths (kept out of the other two: the
// lengths as run-time values cost registers that the softmax threads of the two-group shape do not have).
template <typename T, typename L, int MODE>
__global__ void __launch_bounds__(L::kThreads, 1)
prefill_tc5_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_k_seg,
                   const __grid_constant__ CUtensorMap tm_v_seg, const Tc5Params p) {
    constexpr int NG = L::NG, NB = L::NB, SK = L::kStagesK, SV = L::kStagesV;
    constexpr bool STORE = MODE == 1, RAGGED = MODE == 2;
    constexpr bool kSplitP = sizeof(typename SplitP<T>::yes) != 0 && SplitP<T>::value;
    constexpr int kD = L::D, kKeys = L::KEYS, kTileKV = L::kTileKV, kColTile = L::kColTile;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* k_ring = smem;                                       // tile: two halves [128 keys][64 elements]
    uint8_t* v_ring = k_ring + L::kRingK;
    uint8_t* q_smem = v_ring + L::kRingV;                         // per group two halves [128 rows][64 elements]
    uint64_t* bars = reinterpret_cast<uint64_t*>(q_smem + L::kQ);
    const uint32_t kfull0 = smem_u32(bars), kempty0 = kfull0 + 8 * SK;
    const uint32_t vfull0 = kempty0 + 8 * SK, vempty0 = vfull0 + 8 * SV;
    const uint32_t gbar0 = vempty0 + 8 * SV;                      // group g: +48 g; S buffer 0, S buffer 1, P, O, Q full, Q empty
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kBars);
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nqt = (p.N + kRows * NG - 1) / (kRows * NG);
    const int hb_count = p.H * p.B;
    const int n_items = nqt * hb_count;
    // The CTA's item of round j: the list is sorted longest first and dealt out round-robin; with
    // only a few rounds, in snake order (every other round reversed), which evens out the total
    // length per CTA.
    auto round_item = [&](int j) -> int {
        const int G = (int)gridDim.x, c = (int)blockIdx.x;
        if (p.paired) {
            // Long prompts, many (request, head)s: the query tiles of one (request, head) run at the same
            // time on neighbouring CTAs, so that its K/V crosses HBM once and is found in the L2 by the
            // others (dealt longest-first over all (request, head)s, every query tile re-reads its keys
            // from HBM: 2.3x the unique bytes).  CTA c takes the pr-th longest tile, then the pr-th
            // shortest, of the same (request, head): every CTA gets the same number of key tiles.
            const int ppb = (nqt + 1) / 2;            // CTAs per (request, head)
            const int bpw = G / ppb;                  // (request, head)s in flight
            if (c >= bpw * ppb) return n_items;       // (a few CTAs idle when ppb does not divide the grid)
            const int hb = (j >> 1) * bpw + c / ppb, pr = c % ppb;
            if (hb >= hb_count) return n_items;
            const int qt = (j & 1) ? pr : nqt - 1 - pr;
            if ((j & 1) && 2 * pr == nqt - 1) return n_items;   // the middle tile of an odd count came first
            return (nqt - 1 - qt) * hb_count + hb;
        }
        const int w = j * G + ((p.snake && (j & 1)) ? G - 1 - c : c);
        return w < n_items ? w : n_items;
    };
    // item w -> query tile (longest first), head, request
    auto item_qt = [&](int w) { return nqt - 1 - w / hb_count; };
    // key tiles of group g of query tile qt: up to its diagonal tile (causal); none past the prompt
    // nb = the request's own prompt length: with ragged prompts the items are still laid out for the
    // longest one, and a shorter request leaves its later items (and the tail of one) without work
    auto request_len = [&](int b) -> int { return RAGGED ? __ldg(p.plens + b) : p.N; };
    auto group_tiles = [&](int qt, int g, int nb) -> int {
        const int base = (qt * NG + g) * kRows;
        return base < nb ? min((nb + kKeys - 1) / kKeys, (base + kRows - 1) / kKeys + 1) : 0;
    };

    if (tid == 0) {
        // a stage is released by the MMAs that read it and, when tiles are stored on, by the store thread
        for (int s = 0; s < SK; ++s) {
            mbar_init(kfull0 + 8 * s, 1);
            mbar_init(kempty0 + 8 * s, STORE ? 2 : 1);
        }
        for (int s = 0; s < SV; ++s) {
            mbar_init(vfull0 + 8 * s, 1);
            mbar_init(vempty0 + 8 * s, STORE ? 2 : 1);
        }
        for (int g = 0; g < NG; ++g) {
            mbar_init(gbar0 + 48 * g, 1);
            mbar_init(gbar0 + 48 * g + 8, 1);
            mbar_init(gbar0 + 48 * g + 16, 128);
            mbar_init(gbar0 + 48 * g + 24, 1);
            mbar_init(gbar0 + 48 * g + 32, 1);
            mbar_init(gbar0 + 48 * g + 40, 1);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 4 * NG + 1) {                                     // this warp owns the tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4 * NG) {
        // ------------------------------- TMA producer -------------------------------
        if (lane == 0) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_v);
            auto load_tile = [&](const CUtensorMap* tm, uint8_t* dst_tile, int kt, int kvh, int b, uint32_t full) {
                const uint32_t dst = smem_u32(dst_tile);
                mbar_arrive_expect_tx(full, (uint32_t)kTileKV);
#pragma unroll
                for (int cb = 0; cb < L::kDBoxes; ++cb)
#pragma unroll
                    for (int rb = 0; rb < kKeys / L::kBoxRows; ++rb)
                        tma_load_4d(dst + cb * kColTile + rb * L::kBoxBytes, tm, cb * 64, kvh,
                                    kt * kKeys + rb * L::kBoxRows, b, full);
            };
            uint32_t tp = 0;                                       // K/V tiles requested so far (ring position)
            uint32_t qi[NG];                                      // items group g has taken part in: Q barrier phases
#pragma unroll
            for (int g = 0; g < NG; ++g) qi[g] = 0;
            bool ok = true;
            for (int j = 0; j < p.rounds && ok; ++j) {
                const int w = round_item(j);
                if (w >= n_items) continue;
                const int qt = item_qt(w), hb = w % hb_count, h = hb % p.H, b = hb / p.H;
                const int kvh = h / p.G;
                int nkt = 0;
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    const int gt = group_tiles(qt, g, request_len(b));
                    nkt = max(nkt, gt);
                    if (gt == 0) continue;
                    // the group's Q rows (past the prompt: zeros), once its previous Q is no longer read
                    ok = mbar_wait(gbar0 + 48 * g + 40, (qi[g] & 1) ^ 1, p.wait_ns);
                    if (!ok) break;
                    ++qi[g];
                    const uint32_t qfull = gbar0 + 48 * g + 32;
                    const uint32_t dst = smem_u32(q_smem) + (uint32_t)g * L::kQGroup;
                    mbar_arrive_expect_tx(qfull, (uint32_t)L::kQGroup);
#pragma unroll
                    for (int cb = 0; cb < L::kDBoxes; ++cb)
                        tma_load_4d(dst + cb * kBoxQ, &tm_q, cb * 64, h, (qt * NG + g) * kRows, b, qfull);
                }
                for (int kt = 0; kt < nkt && ok; ++kt, ++tp) {
                    const uint32_t sk = tp % SK, sv = tp % SV;
                    ok = mbar_wait(kempty0 + 8 * sk, ((tp / SK) & 1) ^ 1, p.wait_ns);
                    if (!ok) break;
                    load_tile(&tm_k, k_ring + (size_t)sk * kTileKV, kt, kvh, b, kfull0 + 8 * sk);
                    ok = mbar_wait(vempty0 + 8 * sv, ((tp / SV) & 1) ^ 1, p.wait_ns);
                    if (!ok) break;
                    load_tile(&tm_v, v_ring + (size_t)sv * kTileKV, kt, kvh, b, vfull0 + 8 * sv);
                }
            }
            if (!ok) s_abort = 1;
        } else if (STORE && lane == 1) {
            // ---- fused prefill: the tiles just read from the caller's K/V also become the prompt segment
            // (paper Section 3.2: the prompt is kept once per request).  Tile kt of a kv head is stored by
            // exactly one item: the first query head of the group, at the query tile whose rows start the
            // tile's keys.  The thread follows the producer's tile sequence, waits for a tile to land,
            // stores it if this item owns it (TMA store from the same swizzled tile), and adds its
            // release of the stage to the MMAs' once the store has read shared memory.
            prefetch_tmap(&tm_k_seg);
            prefetch_tmap(&tm_v_seg);
            auto store_tile = [&](const CUtensorMap* tm, uint8_t* src_tile, int kt, int kvh, int b) {
                const uint32_t src = smem_u32(src_tile);
#pragma unroll
                for (int cb = 0; cb < L::kDBoxes; ++cb)
#pragma unroll
                    for (int rb = 0; rb < kKeys / L::kBoxRows; ++rb)
                        tma_store_4d(tm, src + cb * kColTile + rb * L::kBoxBytes, cb * 64, kvh,
                                     kt * kKeys + rb * L::kBoxRows, b);
                bulk_commit_group();
                bulk_wait_read_all();
            };
            uint32_t tp = 0;
            bool ok = true;
            for (int j = 0; j < p.rounds && ok; ++j) {
                const int w = round_item(j);
                if (w >= n_items) continue;
                const int qt = item_qt(w), hb = w % hb_count, h = hb % p.H, b = hb / p.H;
                const int kvh = h / p.G;
                int nkt = 0;
#pragma unroll
                for (int g = 0; g < NG; ++g) nkt = max(nkt, group_tiles(qt, g, request_len(b)));
                for (int kt = 0; kt < nkt && ok; ++kt, ++tp) {
                    const bool mine = (h % p.G) == 0 && (kt * kKeys) / (kRows * NG) == qt;
                    const uint32_t sk = tp % SK, sv = tp % SV;
                    ok = mbar_wait(kfull0 + 8 * sk, (tp / SK) & 1, p.wait_ns);
                    if (!ok) break;
                    if (mine) store_tile(&tm_k_seg, k_ring + (size_t)sk * kTileKV, kt, kvh, b);
                    mbar_arrive(kempty0 + 8 * sk);
                    ok = mbar_wait(vfull0 + 8 * sv, (tp / SV) & 1, p.wait_ns);
                    if (!ok) break;
                    if (mine) store_tile(&tm_v_seg, v_ring + (size_t)sv * kTileKV, kt, kvh, b);
                    mbar_arrive(vempty0 + 8 * sv);
                }
            }
            bulk_wait_all();                                      // the stores themselves, before the CTA may exit
            if (!ok) s_abort = 1;
        }
    } else if (warp == 4 * NG + 1) {
        // -------------------------------- MMA issuer --------------------------------
        if (lane == 0) {
            uint32_t tp = 0;                                       // ring position of the item's first K/V tile
            const uint64_t q_desc0 = smem_desc(smem_u32(q_smem), 16, 1024);
            const uint64_t k_desc0 = smem_desc(smem_u32(k_ring), 16, 1024);
            const uint64_t v_desc0 = smem_desc(smem_u32(v_ring), kColTile, 1024);
            uint32_t n[NG], qi[NG];                               // tiles / items of group g so far: barrier phases
#pragma unroll
            for (int g = 0; g < NG; ++g) n[g] = qi[g] = 0;
            bool ok = true;
            for (int j = 0; j < p.rounds && ok; ++j) {
                const int w = round_item(j);
                if (w >= n_items) continue;
                const int qt = item_qt(w), nb = request_len((w % hb_count) / p.H);
                // requested here, used after the first waits of the item
                const float slope = (kSplitP && p.slopes) ? __ldg(p.slopes + (w % hb_count) % p.H) : 0.f;
                int gt[NG], nkt = 0;
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    gt[g] = group_tiles(qt, g, nb);
                    nkt = max(nkt, gt[g]);
                }
                if (nkt == 0) continue;                           // the request ends before this item's rows
                // S_g[buf] = Q_g . K^T for the group's tile kt; after its last one the group's Q may be replaced
                auto issue_qk = [&](int g, int kt, int buf) {
                    // One descriptor per operand and tile; a K-step only moves the start address, which
                    // sits in the descriptor's low bits in units of 16 bytes: the issuing thread is a
                    // single lane, and every instruction it spends per MMA is time the tensor pipe waits.
                    const uint64_t qd = q_desc0 + (uint64_t)(((uint32_t)g * L::kQGroup) >> 4);
                    const uint64_t kd = k_desc0 + (uint64_t)((((tp + kt) % SK) * (uint32_t)kTileKV) >> 4);
                    const uint32_t d_tmem = tmem + (uint32_t)(kKeys * (g * NB + buf));
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks)
                        tc_mma_ss(d_tmem, qd + (uint64_t)(((ks >> 2) * kBoxQ + (ks & 3) * 32) >> 4),
                                  kd + (uint64_t)(((ks >> 2) * kColTile + (ks & 3) * 32) >> 4), p.idesc_qk, ks > 0);
                    tc_commit(gbar0 + 48 * g + 8 * buf);
                    if (kt + 1 == gt[g]) tc_commit(gbar0 + 48 * g + 40);
                };
                auto wait_k = [&](int kt) -> bool {
                    const bool r = mbar_wait_hot(kfull0 + 8 * ((tp + kt) % SK), ((tp + kt) / SK) & 1, p.wait_ns);
                    tc_fence_after();
                    return r;
                };
#pragma unroll
                for (int g = 0; g < NG; ++g)
                    if (gt[g] > 0 && ok) ok = mbar_wait_hot(gbar0 + 48 * g + 32, qi[g]++ & 1, p.wait_ns);   // Q_g landed
                if (ok) ok = wait_k(0);
                if (!ok) break;
#pragma unroll
                for (int g = 0; g < NG; ++g)
                    if (gt[g] > 0) issue_qk(g, 0, NB == 2 ? (int)(n[g] & 1) : 0);
                tc_commit(kempty0 + 8 * (tp % SK));                // K stage free once these MMAs are done
                for (int kt = 0; kt < nkt && ok; ++kt) {
                    TC5_STAMP(2, kt, 0);
                    if (NB == 2 && kt + 1 < nkt) {                // next tile's scores run under this tile's softmax
                        ok = wait_k(kt + 1);
                        if (!ok) break;
#pragma unroll
                        for (int g = 0; g < NG; ++g)
                            if (kt + 1 < gt[g]) issue_qk(g, kt + 1, (int)((n[g] + 1) & 1));
                        tc_commit(kempty0 + 8 * ((tp + kt + 1) % SK));
                    }
                    const uint32_t sv = (tp + kt) % SV;
                    const uint64_t vd = v_desc0 + (uint64_t)((sv * (uint32_t)kTileKV) >> 4);
                    ok = mbar_wait_hot(vfull0 + 8 * sv, ((tp + kt) / SV) & 1, p.wait_ns);
                    if (!ok) break;
                    bool k_next = false;
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        if (kt >= gt[g]) continue;
                        ok = mbar_wait_hot(gbar0 + 48 * g + 16, n[g] & 1, p.wait_ns);   // P_g written over its S buffer
                        if (!ok) break;
                        TC5_STAMP(2, kt, 1 + 3 * g);
                        tc_fence_after();
                        const uint32_t p_tmem = tmem + (uint32_t)(kKeys * (g * NB + (NB == 2 ? (int)(n[g] & 1) : 0)));
#pragma unroll
                        for (int kk = 0; kk < kKeys / 16; ++kk)   // O_g += P_g[:, 16 keys] . V[16 keys, :]
                            tc_mma_ts(tmem + (uint32_t)(L::kColO + kD * g), p_tmem + kk * 8,
                                      vd + (uint64_t)((kk * 2048) >> 4), p.idesc_pv, (kt > 0 || kk > 0));
                        if (kSplitP && split_p_keys((qt * NG + g) * kRows, kt * kKeys, kKeys, slope)) {
#pragma unroll
                            for (int kk = 0; kk < kKeys / 16; ++kk)   // ... and the low parts of the weights that have one
                                if (split_p_keys((qt * NG + g) * kRows, kt * kKeys + 16 * kk, 16, slope))
                                    tc_mma_ts(tmem + (uint32_t)(L::kColO + kD * g), p_tmem + kKeys / 2 + kk * 8,
                                              vd + (uint64_t)((kk * 2048) >> 4), p.idesc_pv, 1u);
                        }
                        tc_commit(gbar0 + 48 * g + 24);
#if defined(SEGKV_TC5_TIMELINE) && SEGKV_TC5_TIMELINE == 3
                        mbar_wait_hot(gbar0 + 48 * g + 24, n[g] & 1, p.wait_ns);   // measurement only: serialise on P.V
                        TC5_STAMP(2, kt, 2 + 3 * g);
#endif
                        ++n[g];
                        if (NB == 1 && kt + 1 < gt[g]) {          // the group's next scores, behind its P.V in the pipe
                            if (!k_next) {
                                ok = wait_k(kt + 1);
                                if (!ok) break;
                                k_next = true;
                            }
                            issue_qk(g, kt + 1, 0);
#if defined(SEGKV_TC5_TIMELINE) && SEGKV_TC5_TIMELINE == 3
                            mbar_wait_hot(gbar0 + 48 * g, n[g] & 1, p.wait_ns);    // measurement only: serialise on Q.K^T
                            TC5_STAMP(2, kt, 3 + 3 * g);
#endif
                        }
                    }
                    if (!ok) break;
                    tc_commit(vempty0 + 8 * sv);                  // stages free once every MMA so far is done
                    if (NB == 1 && kt + 1 < nkt) tc_commit(kempty0 + 8 * ((tp + kt + 1) % SK));
                }
                tp += (uint32_t)nkt;
            }
            if (!ok) s_abort = 1;
        }
    } else {
        // ------------------------------ softmax warps: one row per thread ------------------------------
        const int g = warp >> 2, r = tid & (kRows - 1);
        const uint32_t bar_s0 = gbar0 + 48 * g, bar_p = bar_s0 + 16, bar_o = bar_s0 + 24;
        const uint32_t tm_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);     // this warp's TMEM lanes
        const uint32_t tm_o = tm_lane + (uint32_t)(L::kColO + kD * g);
        const bool stamp = lane == 0 && (warp & 3) == 0;
        const size_t qstride = (size_t)p.H * kD;
        uint32_t n = 0;                                           // tiles of this group so far: barrier phases
        bool ok = true;
        for (int j = 0; j < p.rounds && ok; ++j) {
            const int w = round_item(j);
            if (w >= n_items) continue;
            const int qt = item_qt(w), hb = w % hb_count, h = hb % p.H, b = hb / p.H;
            const int my_tiles = group_tiles(qt, g, request_len(b));
            if (my_tiles == 0) continue;
            const int row0 = (qt * NG + g) * kRows, row = row0 + r;
            const float slope_nat = p.slopes ? p.slopes[h] : 0.f;
            const float slope2 = slope_nat * 1.4426950408889634f;
            float m_ref = -INFINITY, l_run = 0.f;
            for (int kt = 0; kt < my_tiles; ++kt, ++n) {
                const int buf = NB == 2 ? (int)(n & 1) : 0;
                const uint32_t tm_s = tm_lane + (uint32_t)(kKeys * (g * NB + buf));
                ok = mbar_wait_hot(bar_s0 + 8 * buf, (NB == 2 ? (n >> 1) : n) & 1, p.wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (stamp) TC5_STAMP(g, kt, 0);
                // One tile of the group, from the scores in tensor memory to the weights handed to the
                // MMA thread.  Two instances (weights in one part / in two parts) rather than a branch
                // in the middle: the 128 scores live in registers, and a fork with all of them live
                // costs the two-group shape hundreds of bytes of spills.
                auto tile = [&](auto two_parts) -> bool {
                    constexpr bool split = decltype(two_parts)::value;
                    tc_fence_after();
                    uint32_t sr[kKeys];
#pragma unroll
                    for (int c = 0; c < kKeys / 32; ++c) tc_ld32(tm_s + 32 * c, sr + 32 * c);
                    tc_wait_ld();
                    if (stamp) TC5_STAMP(g, kt, 1);
                    float* sv = reinterpret_cast<float*>(sr);
                    const int key0 = kt * kKeys;
                    const bool diag = key0 + kKeys - 1 > row0;         // a tile that reaches past the group's first row
                    // scores in log2 units: s * scale2 (+ ALiBi bias); the scale is folded into the exponent's
                    // FMA unless a bias has to be added first; keys above the row (diagonal tile) become -inf
                    const bool biased = p.slopes != nullptr;
                    const int lim = row - key0;                        // key index i of this tile is visible iff i <= lim
                    const float bias0 = slope2 * (float)(key0 - row);
                    float tmax;
                    if (biased) tmax = diag ? score_max<kKeys, true, true>(sv, p.scale2, slope2, bias0, lim)
                                            : score_max<kKeys, true, false>(sv, p.scale2, slope2, bias0, lim);
                    else tmax = (diag ? score_max<kKeys, false, true>(sv, p.scale2, slope2, bias0, lim)
                                      : score_max<kKeys, false, false>(sv, p.scale2, slope2, bias0, lim)) * p.scale2;
                    // a new reference only when the maximum has grown by more than 2^8: exponentials stay
                    // below 2^8 of the reference, the sum and O use the same reference
                    const bool need = tmax > m_ref + 8.f;
                    float alpha = 1.f;
                    if (need) {
                        alpha = exp2f(m_ref - tmax);                   // 0 on the first tile
                        m_ref = tmax;
                    }
                    float ls[4] = {0.f, 0.f, 0.f, 0.f};
                    uint32_t pk[kKeys / 2];
                    const float sc = biased ? 1.f : p.scale2, nm = -m_ref;
                    if (!split) {
#pragma unroll
                        for (int i = 0; i < kKeys; i += 2) {
                            const float e0 = exp2f(fmaf(sv[i], sc, nm)), e1 = exp2f(fmaf(sv[i + 1], sc, nm));
                            ls[(i >> 1) & 3] += e0 + e1;
                            pk[i >> 1] = Mma<T>::pack(e0, e1);
                        }
                    } else {
                        // weights as two bf16 parts: the high parts over the first half of the S buffer's
                        // columns, the low parts over the second half, 32 keys at a time (S is in registers
                        // and the MMAs that read the buffer's previous contents have completed)
#pragma unroll
                        for (int c = 0; c < kKeys / 32; ++c) {
                            uint32_t ph[16], pl[16];
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                const float e0 = exp2f(fmaf(sv[32 * c + i], sc, nm)), e1 = exp2f(fmaf(sv[32 * c + i + 1], sc, nm));
                                ls[(i >> 1) & 3] += e0 + e1;
                                const uint32_t b0 = __float_as_uint(e0), b1 = __float_as_uint(e1);
                                ph[i >> 1] = __byte_perm(b0, b1, 0x7632);
                                pl[i >> 1] = Mma<T>::pack(e0 - __uint_as_float(b0 & 0xFFFF0000u), e1 - __uint_as_float(b1 & 0xFFFF0000u));
                            }
                            tc_st16(tm_s + 16 * c, ph);
                            tc_st16(tm_s + kKeys / 2 + 16 * c, pl);
                        }
                    }
                    l_run = l_run * alpha + ((ls[0] + ls[1]) + (ls[2] + ls[3]));
                    if (stamp) TC5_STAMP(g, kt, 2);
                    // O may be touched once P.V of the previous tile is done.  A parity wait is only
                    // meaningful on the barrier's current or previous phase, so with two S buffers,
                    // where nothing else ties this thread to the P.V before last, every phase of the O
                    // barrier is waited for in turn (with one S buffer the scores of this tile were
                    // produced behind that P.V in the pipe, and waiting here is only needed to rescale).
                    const bool rescale = kt > 0 && __any_sync(0xffffffffu, need);
                    if (kt > 0 && (NB == 2 || rescale)) {
                        bool arrived = mbar_wait_hot(bar_o, (n - 1) & 1, p.wait_ns);
                        arrived = __all_sync(0xffffffffu, arrived);
                        if (!arrived) return false;
                        tc_fence_after();
                    }
                    if (rescale) {
#pragma unroll
                        for (int c = 0; c < kD / 32; ++c) {
                            uint32_t orr[32];
                            tc_ld32(tm_o + c * 32, orr);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
                            tc_st32(tm_o + c * 32, orr);
                        }
                        if (stamp) TC5_STAMP(g, kt, 3);
                    }
                    // P over the first 64 columns of the S buffer: two 16-bit weights per column, the A
                    // operand layout of the MMA that follows.  S has been read completely above.
                    if (!split) {
#pragma unroll
                        for (int c = 0; c < kKeys / 32; ++c) tc_st16(tm_s + 16 * c, pk + 16 * c);
                    }
                    tc_wait_st();
                    tc_fence_before();
                    if (!(p.dbg_skip && tid == 0 && n == 0)) mbar_arrive(bar_p);
                    if (stamp) TC5_STAMP(g, kt, 4);
                    return true;
                };
                ok = (kSplitP && split_p_keys(row0, kt * kKeys, kKeys, slope_nat)) ? tile(BoolC<kSplitP>{}) : tile(BoolC<false>{});
                if (!ok) break;
            }
            if (!ok) break;
            // the item's output: O / l, once the last P.V has landed.  The next item's first P.V
            // cannot overwrite O before these loads: it waits for this thread's next P arrival.
            ok = mbar_wait_hot(bar_o, (n - 1) & 1, p.wait_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float inv = 1.f / l_run;
            T* orow = reinterpret_cast<T*>(p.out) + ((size_t)b * p.N * p.H + h) * kD + (size_t)row * qstride;
#pragma unroll
            for (int c = 0; c < kD / 32; ++c) {
                uint32_t orr[32];
                tc_ld32(tm_o + c * 32, orr);
                tc_wait_ld();
                if (row < request_len(b)) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        *reinterpret_cast<uint4*>(orow + c * 32 + i * 8) = make_uint4(
                            Mma<T>::pack(__uint_as_float(orr[8 * i]) * inv, __uint_as_float(orr[8 * i + 1]) * inv),
                            Mma<T>::pack(__uint_as_float(orr[8 * i + 2]) * inv, __uint_as_float(orr[8 * i + 3]) * inv),
                            Mma<T>::pack(__uint_as_float(orr[8 * i + 4]) * inv, __uint_as_float(orr[8 * i + 5]) * inv),
                            Mma<T>::pack(__uint_as_float(orr[8 * i + 6]) * inv, __uint_as_float(orr[8 * i + 7]) * inv));
                }
            }
        }
        if (!ok && lane == 0) s_abort = 1;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4 * NG + 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
        if (lane == 0 && s_abort) atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
    }
}

template <typename T, typename L>
cudaError_t launch_tc5(const Dims& d, const PrefillArgs& a, Tc5Params p, int sms, cudaStream_t st) {
    constexpr int NG = L::NG;
    // Never two CTAs on one SM: each allocates all of tensor memory and keeps it while it walks
    // its items, so a second one would wait for it inside tcgen05.alloc.
    constexpr size_t smem = L::kBytes > 120 * 1024 ? L::kBytes : 120 * 1024;
    static bool configured[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tc5_kernel<T, L, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(prefill_tc5_kernel<T, L, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(prefill_tc5_kernel<T, L, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    // instruction descriptors: fp32 accumulate, A/B format (the same for both operands: a P in fp16
    // against a V in bf16 is not a pair the f16 kind takes), operand majors, N >> 3, M >> 4
    const uint32_t fmt = d.dtype == SEGKV_BF16 ? 1u : 0u;
    const uint32_t common = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kRows >> 4) << 24);
    p.idesc_qk = common | ((uint32_t)(L::KEYS >> 3) << 17);               // A, B both K-major; N = keys of a tile
    p.idesc_pv = common | (1u << 16) | ((uint32_t)(L::D >> 3) << 17);     // B (= V) MN-major; N = head_dim
    p.scale2 = 1.4426950408889634f / sqrtf((float)L::D);
    const long items = (long)((a.prompt_len + kRows * NG - 1) / (kRows * NG)) * d.heads * d.batch;
    const unsigned grid = (unsigned)(items < sms ? items : sms);  // one CTA per SM
    p.snake = items < 8L * sms;
    {
        const int nqt = (a.prompt_len + kRows * NG - 1) / (kRows * NG), ppb = (nqt + 1) / 2;
        const long hb_count = (long)d.heads * d.batch;
        const int bpw = ppb <= sms ? sms / ppb : 0;
        // (not for bf16 with ALiBi, where the two-part weights make the tiles next to the diagonal the
        // expensive ones: measured 20 % slower this way at the Bloom shape, 4 % at twice its prompt)
        const bool two_part_alibi = d.dtype == SEGKV_BF16 && p.slopes != nullptr;
        p.paired = (grid == (unsigned)sms && bpw > 0 && hb_count >= 4L * bpw && !two_part_alibi) ? 1 : 0;
        p.rounds = p.paired ? 2 * (int)((hb_count + bpw - 1) / bpw) : (int)((items + grid - 1) / grid);
    }
    // fused prefill: load through the maps over the caller's arrays, store through the segment's
    const bool store = a.tm_k_src && a.tm_v_src;
    p.store_kv = store ? 1 : 0;
    if (store) prefill_tc5_kernel<T, L, 1><<<grid, L::kThreads, smem, st>>>(*a.tm_q, *a.tm_k_src, *a.tm_v_src, *a.tm_k, *a.tm_v, p);
    else if (p.plens) prefill_tc5_kernel<T, L, 2><<<grid, L::kThreads, smem, st>>>(*a.tm_q, *a.tm_k, *a.tm_v, *a.tm_k, *a.tm_v, p);
    else prefill_tc5_kernel<T, L, 0><<<grid, L::kThreads, smem, st>>>(*a.tm_q, *a.tm_k, *a.tm_v, *a.tm_k, *a.tm_v, p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch_tc5(const Dims& d, const PrefillArgs& a, const Tc5Params& p, int sms, cudaStream_t st) {
    // two row groups per CTA once there are enough 256-row items to fill the machine a few times over
    const long items2 = (long)((a.prompt_len + 2 * kRows - 1) / (2 * kRows)) * d.heads * d.batch;
    const bool two = a.row_groups ? a.row_groups == 2 : items2 >= 2L * sms;
    switch (d.head_dim) {
        case 64:
            return two ? launch_tc5<T, Tc5Layout<64, 128, 2>>(d, a, p, sms, st)
                       : launch_tc5<T, Tc5Layout<64, 128, 1>>(d, a, p, sms, st);
        case 128:
            return two ? launch_tc5<T, Tc5Layout<128, 128, 2>>(d, a, p, sms, st)
                       : launch_tc5<T, Tc5Layout<128, 128, 1>>(d, a, p, sms, st);
        case 256:   // O alone takes 256 of the 512 columns: one group, 64-key tiles, S double-buffered
            return launch_tc5<T, Tc5Layout<256, 64, 1>>(d, a, p, sms, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool prefill_tc5_supported(const Dims& d) { return d.head_dim == 64 || d.head_dim == 128 || d.head_dim == 256; }

cudaError_t launch_prefill_tc5(const Dims& d, const PrefillArgs& a, cudaStream_t st) {
    if (!prefill_tc5_supported(d) || !a.tm_q) return cudaErrorInvalidValue;
    Tc5Params p;
    p.q = a.q; p.out = a.out; p.slopes = a.slopes; p.err_word = a.err_word;
    p.plens = a.plens;
    p.N = a.prompt_len; p.H = d.heads; p.Hkv = d.kv_heads; p.G = d.group; p.B = d.batch;
    p.scale2 = 0.f; p.idesc_qk = p.idesc_pv = 0; p.snake = 0; p.paired = 0; p.rounds = 0;
    p.dbg_skip = a.dbg_skip ? 1 : 0;
    p.wait_ns = a.wait_ns ? a.wait_ns : kWaitLimitNs;
    int sms = 148;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    return d.dtype == SEGKV_BF16 ? dispatch_tc5<__nv_bfloat16>(d, a, p, sms, st) : dispatch_tc5<__half>(d, a, p, sms, st);
}

}  // namespace segkv_impl

#ifdef SEGKV_TC5_TIMELINE
extern "C" __attribute__((visibility("default"))) int segkv_debug_tc5_timeline(long long* host) {
    return cudaMemcpyFromSymbol(host, segkv_impl::g_tc5_tl, sizeof(long long) * 3 * 64 * 8) == cudaSuccess ? 0 : -1;
}
#endif
