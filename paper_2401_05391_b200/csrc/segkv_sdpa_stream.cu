// Persistent form of the fused decode attention (Section 3.3: index selection folded into the
// SDPA kernel; Section 3.2: the prompt segment is read once for all beams of a request).
//
// sdpa_tiled_kernel gives every (request, kv head, split) its own CTA.  When the launch is between one
// and a few waves of CTAs, the last wave is ragged and the SMs that drew no CTA of it idle (wave
// quantisation).  Here a fixed grid of CTAs, two per SM, stays resident and every CTA walks a static
// list of work items (request, kv head, split) dealt round-robin; the split count is chosen by the host
// so that every CTA gets (almost) the same number of items.  Barriers, tensor-map fetches and the
// ring's start-up are paid once per CTA, not once per item, and the producers run ahead into the
// next item while the consumers merge the current one.
//
// Per CTA: CW consumer warps (16 keys of every tile each, as in the tiled kernel), one TMA warp
// (prompt tiles, a ring of RS stages), one gather warp (response rows through the request's list of
// distinct rows, ONE stage of their own; that stage doubles as the scratch of the item's warp merge,
// which is why the gather warp gets it back only after the merge).  Splits are merged through the
// global workspace with an arrival ticket, as in the tiled kernel.  Separate form only (the rows
// come from the list the append kernel made); at most 8 query columns per work group.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "segkv_internal.h"
#include "segkv_ptx.cuh"

namespace segkv_impl {

namespace {

using namespace ptx;

constexpr int kTicketAbortedS = 1 << 16;     // same marker as the tiled kernel's

__device__ __forceinline__ void named_bar(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct StreamParams {
    const void* q;
    void* out;
    const float* slopes;
    const char* kr;                // response K, fixed capacity (V row = K row + vdelta)
    const char* const* k_chunks;   // growing capacity: chunk base pointers, chunk_steps steps each
    long long vdelta;
    const URow* ulist;
    const int32_t* ucount;
    const int32_t* plens;
    float* ws_o;                   // [slab][S][ncols][D]
    float* ws_ml;                  // [slab][S][ncols][2]
    int* tickets;
    int* err_word;
    int P, steps, S, W, G, H, Hkv, rows, max_steps, ncols, RS;
    int chunk_steps, quota, items;
    int early_prompt;              // prompt tiles may be fetched before the previous kernel has completed
    int dbg_skip;
    unsigned long long wait_ns;
    float scale2;
};

// Shared memory (base rounded up to 1024 bytes):
//   RS x {K tile, V tile}     prompt ring, filled by TMA (D/64 boxes of [TILE][128 B], 128B swizzle)
//   1  x {K tile, V tile}     response stage, filled by the gather warp in the same layout;
//                             re-used as the warp-merge scratch of the item's epilogue
//   URow[TILE], row pointers[TILE], mbarriers
template <int D, int CW>
struct StreamLayout {
    static constexpr int TILE = 16 * CW;
    static constexpr int BOX_BYTES = TILE * 128;
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int MERGE_BYTES = CW * 8 * (D + 4 + 2) * 4;
    static_assert(MERGE_BYTES <= STAGE_BYTES, "the warp merge must fit into the response stage");
    static __host__ __device__ constexpr size_t bytes(int rs) {
        return 1024 + (size_t)(rs + 1) * STAGE_BYTES + (size_t)TILE * (sizeof(URow) + 8) + 256;
    }
};

#ifndef SEGKV_STREAM_CTAS
#define SEGKV_STREAM_CTAS 2
#endif
template <typename T, int D, int CW>
__global__ void __launch_bounds__(32 * (CW + 2), SEGKV_STREAM_CTAS)
sdpa_stream_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const StreamParams p) {
    using L = StreamLayout<D, CW>;
    constexpr int TILE = L::TILE;
    constexpr int KS = D / 16;
    constexpr int DP = D + 4;
    constexpr int D4 = D / 4;
    constexpr int CT = CW * 32;
    constexpr int UK = (TILE + 31) / 32;
    constexpr int TMA_WARP = CW, GATHER_WARP = CW + 1;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int RS = p.RS;
    uint8_t* ring = smem;
    uint8_t* rstage = smem + (size_t)RS * L::STAGE_BYTES;
    URow* meta = reinterpret_cast<URow*>(rstage + L::STAGE_BYTES);
    const char** gk = reinterpret_cast<const char**>(meta + TILE);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gk + TILE);
    const uint32_t pfull0 = smem_u32(bars), pempty0 = smem_u32(bars + 8);      // RS <= 8
    const uint32_t rfull = smem_u32(bars + 16), rempty = smem_u32(bars + 17);
    __shared__ int s_last, s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = p.S, ncols = p.ncols;
    int tma_issued = 0;           // TMA warp, lane 0: fills started (for the wind-down after an expired wait)

    // item -> work group and share of it (all roles compute the same thing)
    auto item_of = [&](int it, int& slab, int& split, int& b, int& kvh, int& P, int& pt0, int& pt1) {
        slab = it / S;
        split = it - slab * S;
        b = slab / p.Hkv;
        kvh = slab - b * p.Hkv;
        P = p.plens ? __ldg(p.plens + b) : p.P;
        const int ntp = (P + TILE - 1) / TILE;
        pt0 = (int)((long long)split * ntp / S);
        pt1 = (int)((long long)(split + 1) * ntp / S);
    };

    if (tid == TMA_WARP * 32) {
        for (int s = 0; s < RS; ++s) {
            mbar_init(pfull0 + 8 * s, 1);
            mbar_init(pempty0 + 8 * s, CW);
        }
        mbar_init(rfull, 33);          // every lane of the gather warp (copies landed) plus lane 0 (plain stores)
        mbar_init(rempty, CW);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
    __syncthreads();

    if (warp == TMA_WARP) {
        // =============================== prompt tiles, all items ===============================
        if (lane == 0) {
            if (!p.early_prompt) pdl_wait();
            bool ok = true;
            int kk = 0;                   // tiles issued so far: stage kk % RS, round kk / RS
            for (int it = blockIdx.x; it < p.items && ok; it += gridDim.x) {
                int slab, split, b, kvh, P, pt0, pt1;
                item_of(it, slab, split, b, kvh, P, pt0, pt1);
                for (int t = pt0; t < pt1; ++t, ++kk) {
                    const int st = kk % RS;
                    if (kk >= RS) {
                        ok = mbar_wait(pempty0 + 8 * st, (((uint32_t)(kk / RS)) & 1) ^ 1, p.wait_ns);
                        if (!ok) break;
                    }
                    const uint32_t full = pfull0 + 8 * st;
                    const uint32_t k_dst = smem_u32(ring + (size_t)st * L::STAGE_BYTES);
                    const uint32_t v_dst = k_dst + L::TILE_BYTES;
                    mbar_arrive_expect_tx(full, (uint32_t)L::STAGE_BYTES);
#pragma unroll
                    for (int bx = 0; bx < D / 64; ++bx) {
                        tma_load_4d(k_dst + bx * L::BOX_BYTES, &tm_k, bx * 64, kvh, t * TILE, b, full);
                        tma_load_4d(v_dst + bx * L::BOX_BYTES, &tm_v, bx * 64, kvh, t * TILE, b, full);
                    }
                    tma_issued = kk + 1;
                }
            }
            if (!ok) {
                atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
                s_abort = 1;
            }
            if (p.early_prompt) pdl_wait();
        }
    } else if (warp == GATHER_WARP) {
        // ================= response tiles, all items: index select fused into the load =================
        pdl_wait();
        constexpr int CPR = D / 8;        // 16-byte chunks per row
        constexpr int RPI = 32 / CPR;     // rows covered by one warp-wide copy
        const size_t slab_bytes = (size_t)p.rows * p.Hkv * (size_t)(D * 2);
        auto k_slab = [&](int s) -> const char* {
            if (p.chunk_steps == 0) return p.kr + (size_t)s * slab_bytes;
            const int c = s / p.chunk_steps;
            return p.k_chunks[c] + (size_t)(s - c * p.chunk_steps) * slab_bytes;
        };
        const uint32_t k_dst = smem_u32(rstage), v_dst = k_dst + L::TILE_BYTES;
        const int cap = p.W * p.max_steps;
        bool ok = true;
        int rr = 0;                       // response tiles produced so far
        for (int it = blockIdx.x; it < p.items && ok; it += gridDim.x) {
            int slab, split, b, kvh, P, pt0, pt1;
            item_of(it, slab, split, b, kvh, P, pt0, pt1);
            const URow* ulist_b = p.ulist + (size_t)b * cap;
            const int n_b = p.steps > 0 ? p.ucount[b] : 0;
            const int e0 = min(split * p.quota, n_b);
            const int e1 = (split == S - 1) ? n_b : min((split + 1) * p.quota, n_b);
            const int nrt = max(1, (e1 - e0 + TILE - 1) / TILE);       // every item has a response tile, maybe empty
            for (int r = 0; r < nrt; ++r, ++rr) {
                const int eb = e0 + r * TILE;
                const int cnt = max(0, min(TILE, e1 - eb));
                uint2 u[UK];
#pragma unroll
                for (int kq = 0; kq < UK; ++kq) {
                    const int key = lane + 32 * kq;
                    u[kq] = (key < cnt) ? *reinterpret_cast<const uint2*>(ulist_b + eb + key) : make_uint2(0u, 0u);
                }
                if (rr > 0) {
                    ok = mbar_wait(rempty, ((uint32_t)(rr - 1)) & 1, p.wait_ns);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
#pragma unroll
                for (int kq = 0; kq < UK; ++kq) {
                    const int key = lane + 32 * kq;
                    if (key >= TILE) continue;
                    const bool valid = key < cnt;
                    const int row = valid ? (int)u[kq].x : 0;            // step * rows + slot
                    URow m;
                    m.row = row / p.rows;                                // consumers need the step only
                    m.mask = valid ? u[kq].y : 0u;
                    meta[key] = m;
                    gk[key] = k_slab(m.row) + ((size_t)(row - m.row * p.rows) * p.Hkv + kvh) * (size_t)(D * 2);
                }
                __syncwarp();
                // whole rows per warp-wide copy (CPR lanes per row): coalesced
                const int c = lane % CPR;
                const uint32_t c_off = (uint32_t)(c / 8) * L::BOX_BYTES;
#pragma unroll
                for (int i = 0; i < TILE / RPI; ++i) {
                    if (i * RPI < cnt) {                                  // warp-uniform
                        const int key = i * RPI + lane / CPR;
                        if (key < cnt) {
                            const uint32_t off = c_off + (uint32_t)key * 128 + (uint32_t)(((c & 7) ^ (key & 7)) << 4);
                            const char* src = gk[key] + c * 16;
                            cp_async_16(k_dst + off, src);
                            cp_async_16(v_dst + off, src + p.vdelta);     // a V row sits a constant behind its K row
                        }
                    }
                }
                cp_async_mbar_arrive_noinc(rfull);        // fires when this lane's copies have landed
                // zero the rows between the last real one and the end of its 16-key slice (rows past
                // that slice are never looked at; a masked weight is zero, but zero times whatever
                // bits the stage held before need not be)
                const int fill = min(TILE, (cnt + 15) & ~15);
                const int zchunks = (fill - cnt) * 8;
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx) {
                    uint4* kz = reinterpret_cast<uint4*>(rstage + (size_t)bx * L::BOX_BYTES + (size_t)cnt * 128);
                    uint4* vz = reinterpret_cast<uint4*>(rstage + L::TILE_BYTES + (size_t)bx * L::BOX_BYTES + (size_t)cnt * 128);
                    for (int i = lane; i < zchunks; i += 32) {
                        kz[i] = make_uint4(0u, 0u, 0u, 0u);
                        vz[i] = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                __syncwarp();
                if (lane == 0 && !p.dbg_skip) mbar_arrive(rfull);
            }
        }
        if (!ok && lane == 0) {
            atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            s_abort = 1;
        }
    } else {
        // ======================================= consumer warps =======================================
        pdl_wait();
        pdl_launch_dependents();
        float* mrg_o = reinterpret_cast<float*>(rstage);                 // [CW][8][DP], over the response stage
        float* mrg_ml = mrg_o + (size_t)CW * 8 * DP;                     // [CW][8][2]
        auto chunk_addr = [&](uint32_t base, int key, int ch) -> uint32_t {
            return base + (uint32_t)(ch >> 3) * L::BOX_BYTES + (uint32_t)key * 128 + (uint32_t)(((ch & 7) ^ (key & 7)) << 4);
        };
        bool ok = true;
        int kk = 0, rr = 0;
        int it = blockIdx.x;
        for (; it < p.items; it += gridDim.x) {
            int slab, split, b, kvh, P, pt0, pt1;
            item_of(it, slab, split, b, kvh, P, pt0, pt1);
            // ---- the item's query fragments (Q^T as the B operand: this lane holds column lane/4) ----
            uint32_t qf[KS][2];
            float slope2[2];
            uint32_t beambit[2];
            {
                const int col = lane >> 2;
                const bool cv = col < ncols;
                const int j = cv ? col / p.G : 0, hg = cv ? col % p.G : 0;
                const T* qrow = cv ? reinterpret_cast<const T*>(p.q) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D : nullptr;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int d0 = ks * 16 + (lane & 3) * 2;
                    qf[ks][0] = qrow ? *reinterpret_cast<const uint32_t*>(qrow + d0) : 0u;
                    qf[ks][1] = qrow ? *reinterpret_cast<const uint32_t*>(qrow + d0 + 8) : 0u;
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int col2 = (lane & 3) * 2 + c;
                    const bool cv2 = col2 < ncols;
                    beambit[c] = cv2 ? (1u << (col2 / p.G)) : 0u;
                    slope2[c] = (cv2 && p.slopes) ? p.slopes[kvh * p.G + col2 % p.G] * 1.4426950408889634f : 0.f;
                }
            }
            const int n_b = p.steps > 0 ? p.ucount[b] : 0;
            // the next item's query rows will be wanted in a few microseconds: ask the L2 for them now
            if (it + (int)gridDim.x < p.items && warp == 0) {
                const int slab2 = (it + gridDim.x) / S, b2 = slab2 / p.Hkv, kvh2 = slab2 - b2 * p.Hkv;
                constexpr int LPR = D * 2 / 128;
                for (int i = lane; i < ncols * LPR; i += 32) {
                    const int col = i / LPR;
                    const char* qrow = reinterpret_cast<const char*>(p.q) +
                                       ((size_t)(b2 * p.W + col / p.G) * p.H + kvh2 * p.G + col % p.G) * (size_t)(D * 2);
                    prefetch_l2(qrow + (i % LPR) * 128);
                }
            }
            float o_acc[KS][4];
            float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) o_acc[mt][0] = o_acc[mt][1] = o_acc[mt][2] = o_acc[mt][3] = 0.f;
            const int qpos = P + (p.steps > 0 ? p.steps - 1 : -1);

            // This warp's 16 keys (tile-local kb0 ...) of one tile: scores with the keys on the M side,
            // mask, ALiBi bias, base-2 online softmax, weighted values.
            auto consume = [&](uint32_t k_src, bool resp, int nvalid, int pos0) {
                const int kb0 = warp * 16;
                if (kb0 >= nvalid) return;
                const uint32_t v_src = k_src + L::TILE_BYTES;
                float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t a[4];
                    ldmatrix_x4(a, chunk_addr(k_src, kb0 + (lane & 15), 2 * ks + (lane >> 4)));
                    Mma<T>::run(sc, a, qf[ks][0], qf[ks][1]);
                }
                uint32_t kmask[2];
                float kpos[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int key = kb0 + (lane >> 2) + 8 * r;
                    if (resp) {
                        const URow u = meta[key];                        // {step, beams that read the row}
                        kmask[r] = key < nvalid ? u.mask : 0u;
                        kpos[r] = (float)(P + u.row - qpos);
                    } else {
                        kmask[r] = key < nvalid ? 0xffffffffu : 0u;
                        kpos[r] = (float)(pos0 + key - qpos);
                    }
                }
                // bf16 keeps 8 significant bits of a weight: such weights go to the tensor cores in two
                // parts (hi + lo); the kernel is bound by HBM and the second set of MMAs is free
                constexpr bool kTwoPart = !Mma<T>::kWeights11Bits;
                float s[2][2];
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const float v = sc[2 * r + c] * p.scale2 + slope2[c] * kpos[r];
                        s[r][c] = (kmask[r] & beambit[c]) ? v : -INFINITY;
                    }
                bool rescale = false;
                float alpha[2];
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float tm = fmaxf(s[0][c], s[1][c]);
                    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 4));
                    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 8));
                    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 16));
                    const float m_old = m_run[c];
                    const float m_new = fmaxf(m_old, tm);
                    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                    const float a = exp2f(m_old - m_use);
                    alpha[c] = a;
                    rescale = rescale || (a != 1.f);
                    m_run[c] = m_new;
                    const float p0 = exp2f(s[0][c] - m_use), p1 = exp2f(s[1][c] - m_use);
                    s[0][c] = p0;
                    s[1][c] = p1;
                    l_run[c] = l_run[c] * a + p0 + p1;
                }
                const uint32_t h0 = Mma<T>::pack(s[0][0], s[0][1]), h1 = Mma<T>::pack(s[1][0], s[1][1]);
                const uint32_t pf0 = movmatrix_trans(h0), pf1 = movmatrix_trans(h1);
                uint32_t pl0 = 0, pl1 = 0;
                if constexpr (kTwoPart) {
                    pl0 = movmatrix_trans(Mma<T>::pack(s[0][0] - __uint_as_float(h0 << 16), s[0][1] - __uint_as_float(h0 & 0xFFFF0000u)));
                    pl1 = movmatrix_trans(Mma<T>::pack(s[1][0] - __uint_as_float(h1 << 16), s[1][1] - __uint_as_float(h1 & 0xFFFF0000u)));
                }
                if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        o_acc[mt][0] *= alpha[0];
                        o_acc[mt][1] *= alpha[1];
                        o_acc[mt][2] *= alpha[0];
                        o_acc[mt][3] *= alpha[1];
                    }
                }
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, chunk_addr(v_src, kb0 + (lane & 7) + 8 * (lane >> 4), 2 * mt + ((lane >> 3) & 1)));
                    Mma<T>::run(o_acc[mt], a, pf0, pf1);
                    if constexpr (kTwoPart) Mma<T>::run(o_acc[mt], a, pl0, pl1);
                }
            };

            // ---- prompt tiles ----
            for (int t = pt0; t < pt1; ++t, ++kk) {
                const int st = kk % RS;
                ok = mbar_wait(pfull0 + 8 * st, ((uint32_t)(kk / RS)) & 1, p.wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                consume(smem_u32(ring + (size_t)st * L::STAGE_BYTES), false, min(TILE, P - t * TILE), t * TILE);
                __syncwarp();
                if (lane == 0) mbar_arrive(pempty0 + 8 * st);
            }
            if (!ok) break;
            // ---- response tiles (the last one's stage is kept for the merge below) ----
            const int e0 = min(split * p.quota, n_b);
            const int e1 = (split == S - 1) ? n_b : min((split + 1) * p.quota, n_b);
            const int nrt = max(1, (e1 - e0 + TILE - 1) / TILE);
            for (int r = 0; r < nrt; ++r, ++rr) {
                ok = mbar_wait(rfull, ((uint32_t)rr) & 1, p.wait_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                consume(smem_u32(rstage), true, max(0, min(TILE, e1 - (e0 + r * TILE))), 0);
                __syncwarp();
                if (r < nrt - 1 && lane == 0) mbar_arrive(rempty);
            }
            if (!ok) break;

            // ---- merge the consumer warps (each saw a different quarter of every tile) ----
            named_bar(1, CT);                             // every consumer warp is done reading the stage
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                float l = l_run[c];
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                const int col = (lane & 3) * 2 + c;
                if ((lane >> 2) == 0) {
                    mrg_ml[((size_t)warp * 8 + col) * 2 + 0] = m_run[c];
                    mrg_ml[((size_t)warp * 8 + col) * 2 + 1] = l;
                }
                float* dst = mrg_o + ((size_t)warp * 8 + col) * DP + (lane >> 2);
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    dst[mt * 16] = o_acc[mt][c];
                    dst[mt * 16 + 8] = o_acc[mt][2 + c];
                }
            }
            named_bar(1, CT);
            auto store_out = [&](int col, int d, float4 o) {
                const int j = col / p.G, hg = col % p.G;
                T* orow = reinterpret_cast<T*>(p.out) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D + d;
                uint2 pk;
                pk.x = Mma<T>::pack(o.x, o.y);
                pk.y = Mma<T>::pack(o.z, o.w);
                *reinterpret_cast<uint2*>(orow) = pk;
            };
            float* wso_it = p.ws_o + (size_t)it * ncols * D;             // it = slab * S + split
            float* wsml_it = p.ws_ml + (size_t)it * ncols * 2;
            for (int x = tid; x < ncols * D4; x += CT) {
                const int col = x / D4, d = (x % D4) * 4;
                float mm = -INFINITY;
#pragma unroll
                for (int w = 0; w < CW; ++w) mm = fmaxf(mm, mrg_ml[((size_t)w * 8 + col) * 2]);
                float ll = 0.f;
                float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < CW; ++w) {
                    const float mw = mrg_ml[((size_t)w * 8 + col) * 2];
                    const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - mm);
                    ll += mrg_ml[((size_t)w * 8 + col) * 2 + 1] * f;
                    const float4 v = *reinterpret_cast<const float4*>(mrg_o + ((size_t)w * 8 + col) * DP + d);
                    o.x += v.x * f; o.y += v.y * f; o.z += v.z * f; o.w += v.w * f;
                }
                if (S == 1) {
                    const float inv = 1.f / ll;
                    o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
                    store_out(col, d, o);
                } else {
                    *reinterpret_cast<float4*>(wso_it + (size_t)col * D + d) = o;
                    if (d == 0) *reinterpret_cast<float2*>(wsml_it + col * 2) = make_float2(mm, ll);
                }
            }
            if (S > 1) {
                // the last CTA of the work group to arrive (atomic ticket, nobody waits) merges all partials
                named_bar(1, CT);
                if (tid == 0) {
                    int ticket;
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(ticket) : "l"(p.tickets + slab) : "memory");
                    s_last = (ticket & (kTicketAbortedS - 1)) == S - 1 ? 1 + (ticket >= kTicketAbortedS ? 1 : 0) : 0;
                    if (s_last == 2) p.tickets[slab] = 0;     // a CTA of the group gave up: no merge, counter ready for the next launch
                }
                named_bar(1, CT);
                if (s_last == 1) {
                    const float2* wsml_slab = reinterpret_cast<const float2*>(p.ws_ml + (size_t)slab * S * ncols * 2);
                    const float* wso_slab = p.ws_o + (size_t)slab * S * ncols * D;
                    for (int x = tid; x < ncols * D4; x += CT) {
                        const int col = x / D4, d = (x % D4) * 4;
                        const float4* src = reinterpret_cast<const float4*>(wso_slab + (size_t)col * D + d);
                        const size_t sstride = (size_t)ncols * D4;
                        float mm = -INFINITY, ll = 0.f;
                        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int s0 = 0; s0 < S; s0 += 4) {
                            float4 v[4];
                            float2 ml[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const bool in = s0 + u < S;
                                ml[u] = in ? __ldcg(wsml_slab + (size_t)(s0 + u) * ncols + col) : make_float2(-INFINITY, 0.f);
                                v[u] = in ? __ldcg(src + (size_t)(s0 + u) * sstride) : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
                            float bm = mm;
#pragma unroll
                            for (int u = 0; u < 4; ++u) bm = fmaxf(bm, ml[u].x);
                            const float fo = (mm == -INFINITY) ? 0.f : exp2f(mm - bm);
                            ll *= fo; o.x *= fo; o.y *= fo; o.z *= fo; o.w *= fo;
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
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
                }
            }
            // the scratch is free again: the gather warp may fill the stage for the next item
            named_bar(1, CT);
            if (lane == 0) mbar_arrive(rempty);
        }
        if (!ok) {
            if (lane == 0) {
                atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
                s_abort = 1;
            }
            // The arrival counters of the work groups must still come back to zero for the next launch:
            // take the ticket of this and every later item of this CTA, marked, so that the last arriver
            // of each group skips the merge (its output stays untouched).
            if (S > 1 && tid == 0) {
                for (; it < p.items; it += gridDim.x) {
                    const int slab = it / S;
                    int ticket;
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(ticket) : "l"(p.tickets + slab), "r"(kTicketAbortedS + 1) : "memory");
                    if ((ticket & (kTicketAbortedS - 1)) == S - 1) p.tickets[slab] = 0;
                }
            }
        }
    }
    // The CTA leaves together.  After an expired wait, copies still in flight get a bounded chance to
    // land before the shared memory is released.
    __syncthreads();
    if (s_abort != 0) {
        if (warp == TMA_WARP && lane == 0)
            for (int k = max(0, tma_issued - RS); k < tma_issued; ++k)
                (void)mbar_wait(pfull0 + 8 * (k % RS), ((uint32_t)(k / RS)) & 1, p.wait_ns);
        if (warp == GATHER_WARP) cp_async_wait_all();
    }
}

template <typename T, int D, int CW>
cudaError_t launch_stream_one(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv,
                              int sm_count, cudaStream_t st) {
    using L = StreamLayout<D, CW>;
    // prompt ring: what two CTAs per SM leave room for, at most 8 stages
    int rs = (int)(((SEGKV_STREAM_CTAS == 1 ? 224 : 110) * 1024 - 1024 - 256 - L::TILE * 16) / L::STAGE_BYTES) - 1;
    if (rs > 8) rs = 8;
    if (rs < 1) return cudaErrorInvalidValue;
    const size_t smem = L::bytes(rs);
    auto kern = sdpa_stream_kernel<T, D, CW>;
    static size_t configured[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && configured[dev] < smem) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = smem;
    }
    StreamParams p;
    p.q = a.q; p.out = a.out; p.slopes = a.slopes;
    p.kr = (const char*)a.kr; p.k_chunks = (const char* const*)a.k_chunks; p.vdelta = a.vdelta;
    p.chunk_steps = d.chunk_steps;
    p.ulist = a.ulist; p.ucount = a.ucount; p.plens = a.plens;
    p.tickets = a.tickets; p.err_word = a.err_word;
    p.P = a.prompt_len; p.steps = a.steps; p.S = a.splits; p.W = d.beams; p.G = d.group; p.H = d.heads;
    p.Hkv = d.kv_heads; p.rows = d.rows; p.max_steps = d.max_steps; p.ncols = d.beams * d.group; p.RS = rs;
    p.scale2 = 1.4426950408889634f / sqrtf((float)D);
    p.quota = (a.steps + 2 * d.beams + a.splits - 1) / a.splits;      // the tiled kernel's rule
    if (p.quota < 1) p.quota = 1;
    const size_t slabs = (size_t)d.batch * d.kv_heads;
    p.items = (int)(slabs * a.splits);
    p.early_prompt = (a.pdl && a.prompt_immutable) ? 1 : 0;
    p.dbg_skip = a.dbg_skip ? 1 : 0;
    p.wait_ns = a.wait_ns ? a.wait_ns : kWaitLimitNs;
    p.ws_o = a.ws;
    p.ws_ml = a.ws ? a.ws + slabs * a.splits * p.ncols * D : nullptr;

    cudaLaunchConfig_t cfg = {};
    const int grid = p.items < SEGKV_STREAM_CTAS * sm_count ? p.items : SEGKV_STREAM_CTAS * sm_count;
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(32 * (CW + 2), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    unsigned na = 0;
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
cudaError_t stream_dispatch(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv,
                            int sm_count, cudaStream_t st) {
    switch (d.head_dim) {
        case 64: return launch_stream_one<T, 64, 4>(d, a, tmk, tmv, sm_count, st);
        case 128: return launch_stream_one<T, 128, 4>(d, a, tmk, tmv, sm_count, st);
        case 256: return launch_stream_one<T, 256, 2>(d, a, tmk, tmv, sm_count, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool stream_supported(const Dims& d) {
    return d.beams * d.group <= 8 && (d.head_dim == 64 || d.head_dim == 128 || d.head_dim == 256);
}

// Persistent CTAs resident per SM (what the grid is sized for).
int stream_ctas_per_sm() { return SEGKV_STREAM_CTAS; }

// Takes the tensor maps of the regular tile shape (64-key boxes; 32-key boxes at head_dim 256).
// a.splits: items per work group; the workspace and tickets as for the tiled kernel's workspace merge.
cudaError_t launch_sdpa_stream(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv,
                               int sm_count, cudaStream_t st) {
    if (!stream_supported(d) || a.fused || a.splits < 1) return cudaErrorInvalidValue;
    return d.dtype == SEGKV_BF16 ? stream_dispatch<__nv_bfloat16>(d, a, tmk, tmv, sm_count, st)
                                 : stream_dispatch<__half>(d, a, tmk, tmv, sm_count, st);
}

}  // namespace segkv_impl
