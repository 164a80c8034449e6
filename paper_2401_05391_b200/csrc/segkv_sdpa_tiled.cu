// Tiled split-KV decode attention for sm_100a.
//
// What it computes: paper Section 3.3 ("Customized SDPA Kernel") — for each
// (request, kv head) work group the query block Q[BW, D] attends to the shared
// prompt K/V [N_prompt, D] and to the index-selected response rows, with one
// softmax over both parts.  How it is organised here is specific to B200:
//
//  * grid = (request, kv head, split).  A CTA owns ALL beams (and all query
//    heads of the kv head's group) of its work group, so a K/V byte staged in
//    shared memory is used by every beam: prompt bytes cross HBM once, not BW
//    times (Section 4.2.1: "accesses only 1/BW amount data in HBM").
//  * one producer warp feeds a ring of shared-memory stages.  Prompt tiles come
//    by TMA (cp.async.bulk.tensor, 128-byte swizzle) from the head-major prompt
//    segment; response tiles are gathered row by row with 16-byte cp.async
//    through the request's list of DISTINCT response rows (the index select of
//    Section 3.3 folded into the load), written into the same swizzled layout.
//    Every row carries the set of beams that read it; scores of other beams
//    are masked, so a row shared by several beams is also fetched once.
//  * consumer warps take 16 keys of a tile each.  Scores are a small GEMM on
//    tensor cores with the KEYS on the M side: S^T[16 keys, 8 cols] = K . Q^T
//    (mma.sync m16n8k16, fp32 accumulate), so the BW=4 beams pad only to 8.
//    Online softmax in fp32 (base-2 exponent), P^T transposed in registers
//    (movmatrix) and O^T[16 d, 8 cols] += V^T . P^T, V^T read with
//    ldmatrix.trans.  Each warp keeps its own running max / sum / O^T.
//  * epilogue: warps merge through shared memory; with more than one split the
//    partial (m, l, O) goes to a workspace and the last CTA of the work group
//    to arrive (atomic ticket, no waiting) merges the splits and writes out.
//
// All mbarrier waits are bounded: on expiry the kernel sets
// SEGKV_DEV_WAIT_LIMIT in the error word and winds down.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "segkv_internal.h"

namespace segkv_impl {

namespace {

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait (about two seconds): false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > 2000000000ull) return false;
    }
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(m), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_8(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_mbar_arrive_noinc(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

template <typename T> struct Mma;
template <> struct Mma<__half> {
    static __device__ __forceinline__ void run(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&h);
    }
    static __device__ __forceinline__ __half down(float f) { return __float2half_rn(f); }
};
template <> struct Mma<__nv_bfloat16> {
    static __device__ __forceinline__ void run(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&h);
    }
    static __device__ __forceinline__ __nv_bfloat16 down(float f) { return __float2bfloat16_rn(f); }
};

struct TiledParams {
    const void* q;
    void* out;
    const float* slopes;
    const char* kr;
    const char* vr;
    const URow* ulist;
    const int32_t* ucount;
    float* ws;
    int* tickets;
    int* err_word;
    int P, steps, S, W, G, H, Hkv, rows, max_steps, ncols, stages;
    float scale2;  // log2(e) / sqrt(D)
};

// Shared-memory carve-up (after rounding the base up to 1024 bytes):
//   stages x { K tile, V tile }      each tile = D/64 boxes of [TILE rows][128 B], 128B-swizzled
//   stages x URow[TILE]              per-key row id and beam mask of response tiles
//   full[stages], empty[stages]      mbarriers
// The warp-merge buffer of the epilogue re-uses the stage area.
template <int D, int CW>
struct Layout {
    static constexpr int TILE = 16 * CW;
    static constexpr int BOX_BYTES = TILE * 128;
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int META_BYTES = TILE * (int)sizeof(URow);
    static __host__ __device__ constexpr size_t bytes(int stages, int nt) {
        size_t ring = (size_t)stages * (STAGE_BYTES + META_BYTES);
        size_t merge = (size_t)CW * 8 * nt * (D + 4 + 2) * 4;
        size_t body = ring > merge ? ring : merge;
        return 1024 + body + (size_t)stages * 16 + 64;
    }
};

template <typename T, int D, int NT, int CW>
__global__ void __launch_bounds__(32 * (CW + 1), NT > 1 ? 1 : 2)
sdpa_tiled_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const TiledParams p) {
    using L = Layout<D, CW>;
    constexpr int TILE = L::TILE;
    constexpr int KS = D / 16;           // k-steps of Q.K, m-tiles of P.V
    constexpr int NTHREADS = 32 * (CW + 1);
    constexpr int DP = D + 4;            // padded row of the merge buffer (conflict-free)

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stages = p.stages;
    uint8_t* ring = smem;
    URow* meta = reinterpret_cast<URow*>(ring + (size_t)stages * L::STAGE_BYTES);
    size_t ring_bytes = (size_t)stages * (L::STAGE_BYTES + L::META_BYTES);
    size_t merge_bytes = (size_t)CW * 8 * NT * (DP + 2) * 4;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (ring_bytes > merge_bytes ? ring_bytes : merge_bytes));
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + stages);
    __shared__ int s_last, s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x % p.S;
    const int slab = blockIdx.x / p.S;           // b * Hkv + kvh
    const int b = slab / p.Hkv, kvh = slab % p.Hkv;

    // this CTA's share: whole prompt tiles, and a range of the request's distinct response rows
    const int ntp = (p.P + TILE - 1) / TILE;
    const int pt0 = (int)((long long)split * ntp / p.S), pt1 = (int)((long long)(split + 1) * ntp / p.S);
    const int n_b = p.steps > 0 ? p.ucount[b] : 0;
    const int e0 = (int)((long long)split * n_b / p.S), e1 = (int)((long long)(split + 1) * n_b / p.S);
    const int npt = pt1 - pt0;
    const int nrt = (e1 - e0 + TILE - 1) / TILE;
    const int ntiles = npt + nrt;
    const URow* ulist_b = p.ulist + (size_t)b * p.W * p.max_steps;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full0 + 8 * s, 32);     // every producer lane arrives once per fill
            mbar_init(empty0 + 8 * s, CW);    // one arrival per consumer warp
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();

    // consumer state (declared here so that the epilogue sees it)
    float o_acc[NT][KS][4];
    float m_run[NT][2], l_run[NT][2];

    if (warp == CW) {
        // ================================ producer warp ================================
        if (lane == 0 && npt > 0) {
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_v);
        }
        bool ok = true;
        for (int k = 0; k < ntiles && ok; ++k) {
            const int st = k % stages;
            const uint32_t round = (uint32_t)(k / stages);
            ok = mbar_wait(empty0 + 8 * st, (round & 1) ^ 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t full = full0 + 8 * st;
            const uint32_t k_dst = smem_u32(ring + (size_t)st * L::STAGE_BYTES);
            const uint32_t v_dst = k_dst + L::TILE_BYTES;
            if (k < npt) {
                if (lane == 0) {
                    mbar_arrive_expect_tx(full, (uint32_t)L::STAGE_BYTES);
                    const int y = (pt0 + k) * TILE;
#pragma unroll
                    for (int bx = 0; bx < D / 64; ++bx) {
                        tma_load_3d(k_dst + bx * L::BOX_BYTES, &tm_k, bx * 64, y, slab, full);
                        tma_load_3d(v_dst + bx * L::BOX_BYTES, &tm_v, bx * 64, y, slab, full);
                    }
                } else {
                    mbar_arrive(full);
                }
            } else {
                const int eb = e0 + (k - npt) * TILE;
                const int cnt = min(TILE, e1 - eb);
                const uint32_t meta_dst = smem_u32(meta + (size_t)st * TILE);
                constexpr int UK = (TILE + 31) / 32;
                int urow[UK];
#pragma unroll
                for (int kk = 0; kk < UK; ++kk) {
                    const int key = lane + 32 * kk;
                    urow[kk] = 0;
                    if (key < TILE) {
                        const bool valid = key < cnt;
                        if (valid) urow[kk] = ulist_b[eb + key].row;
                        cp_async_8(meta_dst + key * 8, valid ? (const void*)(ulist_b + eb + key) : (const void*)p.ulist,
                                   valid ? 8u : 0u);
                    }
                }
                constexpr int CPR = D / 8;        // 16-byte chunks per row
                constexpr int RPI = 32 / CPR;     // rows covered by one warp-wide copy
                const int c = lane % CPR;
                const uint32_t c_off = (uint32_t)(c / 8) * L::BOX_BYTES;
#pragma unroll 4
                for (int i = 0; i < TILE / RPI; ++i) {
                    const int key = i * RPI + lane / CPR;
                    int r = urow[0];
                    if (TILE > 32 && key >= 32) r = urow[UK - 1];
                    r = __shfl_sync(0xffffffffu, r, key & 31);
                    const bool valid = key < cnt;
                    const size_t src = ((size_t)r * p.Hkv + kvh) * (size_t)(D * 2) + (size_t)c * 16;
                    const uint32_t off = c_off + (uint32_t)key * 128 + (uint32_t)(((c & 7) ^ (key & 7)) << 4);
                    cp_async_16(k_dst + off, valid ? p.kr + src : p.kr, valid ? 16u : 0u);
                    cp_async_16(v_dst + off, valid ? p.vr + src : p.vr, valid ? 16u : 0u);
                }
                cp_async_mbar_arrive_noinc(full);
            }
        }
        if (!ok && lane == 0) {
            atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            s_abort = 1;
        }
    } else {
        // ================================ consumer warps ===============================
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            m_run[nt][0] = m_run[nt][1] = -INFINITY;
            l_run[nt][0] = l_run[nt][1] = 0.f;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) o_acc[nt][mt][i] = 0.f;
        }
        // Q^T as the B operand: this lane holds column n = lane/4 of every column tile
        uint32_t qf[NT][KS][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int col = nt * 8 + (lane >> 2);
            const bool cv = col < p.ncols;
            const int j = cv ? col / p.G : 0, hg = cv ? col % p.G : 0;
            const T* qrow = reinterpret_cast<const T*>(p.q) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const int d0 = ks * 16 + (lane & 3) * 2;
                qf[nt][ks][0] = cv ? *reinterpret_cast<const uint32_t*>(qrow + d0) : 0u;
                qf[nt][ks][1] = cv ? *reinterpret_cast<const uint32_t*>(qrow + d0 + 8) : 0u;
            }
        }
        // the two score columns this lane owns in every column tile
        float slope2[NT][2];
        uint32_t beambit[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int col = nt * 8 + (lane & 3) * 2 + c;
                const bool cv = col < p.ncols;
                beambit[nt][c] = cv ? (1u << (col / p.G)) : 0u;
                slope2[nt][c] = (cv && p.slopes) ? p.slopes[kvh * p.G + col % p.G] * 1.4426950408889634f : 0.f;
            }
        const int qpos = p.P + (p.steps > 0 ? p.steps - 1 : -1);
        const int key_lo = warp * 16 + (lane >> 2);       // tile-local key of accumulator rows 0..7

        bool ok = true;
        for (int k = 0; k < ntiles; ++k) {
            const int st = k % stages;
            const uint32_t round = (uint32_t)(k / stages);
            ok = mbar_wait(full0 + 8 * st, round & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t k_src = smem_u32(ring + (size_t)st * L::STAGE_BYTES);
            const uint32_t v_src = k_src + L::TILE_BYTES;
            const bool resp = k >= npt;
            int nvalid;        // keys of this tile that exist
            if (!resp) nvalid = min(TILE, p.P - (pt0 + k) * TILE);
            else nvalid = min(TILE, e1 - (e0 + (k - npt) * TILE));

            if (warp * 16 < nvalid) {
                // ---- S^T = K . Q^T ----
                float sc[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
                {
                    const int key = warp * 16 + (lane & 15);
                    const uint32_t rowaddr = k_src + (uint32_t)key * 128;
                    const int sw = key & 7;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int ch = 2 * ks + (lane >> 4);
                        uint32_t a[4];
                        ldmatrix_x4(a, rowaddr + (uint32_t)(ch >> 3) * L::BOX_BYTES + (uint32_t)(((ch & 7) ^ sw) << 4));
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) Mma<T>::run(sc[nt], a, qf[nt][ks][0], qf[nt][ks][1]);
                    }
                }
                // ---- mask, bias, online softmax ----
                uint32_t kmask[2];
                float kpos[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int key = key_lo + 8 * r;
                    if (resp) {
                        const URow u = meta[(size_t)st * TILE + key];
                        kmask[r] = u.mask;                      // zero for padding rows
                        kpos[r] = (float)(p.P + u.row / p.rows - qpos);
                    } else {
                        kmask[r] = key < nvalid ? 0xffffffffu : 0u;
                        kpos[r] = (float)((pt0 + k) * TILE + key - qpos);
                    }
                }
                uint32_t pfrag[NT][2];
                bool rescale = false;
                float alpha[NT][2];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    float s[2][2];
#pragma unroll
                    for (int r = 0; r < 2; ++r)
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            float v = sc[nt][2 * r + c] * p.scale2 + slope2[nt][c] * kpos[r];
                            s[r][c] = (kmask[r] & beambit[nt][c]) ? v : -INFINITY;
                        }
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        float tm = fmaxf(s[0][c], s[1][c]);
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
                        const float p0 = exp2f(s[0][c] - m_use), p1 = exp2f(s[1][c] - m_use);
                        s[0][c] = p0;
                        s[1][c] = p1;
                        l_run[nt][c] = l_run[nt][c] * a + p0 + p1;
                    }
                    // P^T as the B operand of O^T += V^T . P^T
                    pfrag[nt][0] = movmatrix_trans(Mma<T>::pack(s[0][0], s[0][1]));
                    pfrag[nt][1] = movmatrix_trans(Mma<T>::pack(s[1][0], s[1][1]));
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
                {
                    const int key = warp * 16 + (lane & 7) + 8 * (lane >> 4);
                    const uint32_t rowaddr = v_src + (uint32_t)key * 128;
                    const int sw = key & 7;
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        const int ch = 2 * mt + ((lane >> 3) & 1);
                        uint32_t a[4];
                        ldmatrix_x4_trans(a, rowaddr + (uint32_t)(ch >> 3) * L::BOX_BYTES + (uint32_t)(((ch & 7) ^ sw) << 4));
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) Mma<T>::run(o_acc[nt][mt], a, pfrag[nt][0], pfrag[nt][1]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * st);
        }
        if (!ok && lane == 0) {
            atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
            s_abort = 1;
        }
    }

    // ==================================== epilogue ====================================
    __syncthreads();
    if (s_abort) {
        // Something never arrived.  Give copies still in flight a bounded chance to land
        // before the shared memory is released, then leave without touching the output.
        if (warp == CW && lane == 0)
            for (int k = max(0, ntiles - stages); k < ntiles; ++k)
                (void)mbar_wait(full0 + 8 * (k % stages), (uint32_t)(k / stages) & 1);
        return;
    }

    float* mrg_o = reinterpret_cast<float*>(smem);                       // [CW][8*NT][DP]
    float* mrg_ml = mrg_o + (size_t)CW * 8 * NT * DP;                    // [CW][8*NT][2]
    if (warp < CW) {
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
    float* ws_cta = p.ws + ((size_t)slab * p.S + split) * ncols * (D + 2);
    for (int idx = tid; idx < ncols * D; idx += NTHREADS) {
        const int col = idx / D, d = idx % D;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < CW; ++w) mm = fmaxf(mm, mrg_ml[((size_t)w * 8 * NT + col) * 2]);
        float ll = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < CW; ++w) {
            const float mw = mrg_ml[((size_t)w * 8 * NT + col) * 2];
            const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - mm);
            ll += mrg_ml[((size_t)w * 8 * NT + col) * 2 + 1] * f;
            o += mrg_o[((size_t)w * 8 * NT + col) * DP + d] * f;
        }
        if (p.S == 1) {
            const int j = col / p.G, hg = col % p.G;
            T* orow = reinterpret_cast<T*>(p.out) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D;
            orow[d] = Mma<T>::down(o / ll);
        } else {
            ws_cta[(size_t)col * (D + 2) + d] = o;
            if (d == 0) {
                ws_cta[(size_t)col * (D + 2) + D] = mm;
                ws_cta[(size_t)col * (D + 2) + D + 1] = ll;
            }
        }
    }
    if (p.S == 1) return;

    // ---- split merge by the last CTA of this work group to arrive ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(p.tickets + slab, 1);
        s_last = (ticket == p.S - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const float* ws_slab = p.ws + (size_t)slab * p.S * ncols * (D + 2);
    for (int idx = tid; idx < ncols * D; idx += NTHREADS) {
        const int col = idx / D, d = idx % D;
        float mm = -INFINITY;
        for (int s = 0; s < p.S; ++s) mm = fmaxf(mm, __ldcg(ws_slab + ((size_t)s * ncols + col) * (D + 2) + D));
        float ll = 0.f, o = 0.f;
        for (int s = 0; s < p.S; ++s) {
            const float* part = ws_slab + ((size_t)s * ncols + col) * (D + 2);
            const float ms = __ldcg(part + D);
            const float f = (ms == -INFINITY) ? 0.f : exp2f(ms - mm);
            ll += __ldcg(part + D + 1) * f;
            o += __ldcg(part + d) * f;
        }
        const int j = col / p.G, hg = col % p.G;
        T* orow = reinterpret_cast<T*>(p.out) + ((size_t)(b * p.W + j) * p.H + kvh * p.G + hg) * D;
        orow[d] = Mma<T>::down(o / ll);
    }
    if (tid == 0) p.tickets[slab] = 0;      // ready for the next launch
}

template <typename T, int D, int NT, int CW>
cudaError_t launch_one(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv, int stages,
                       cudaStream_t st) {
    using L = Layout<D, CW>;
    const size_t smem = L::bytes(stages, NT);
    auto kern = sdpa_tiled_kernel<T, D, NT, CW>;
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
    p.kr = (const char*)a.kr; p.vr = (const char*)a.vr;
    p.ulist = a.ulist; p.ucount = a.ucount; p.ws = a.ws; p.tickets = a.tickets; p.err_word = a.err_word;
    p.P = a.prompt_len; p.steps = a.steps; p.S = a.splits; p.W = d.beams; p.G = d.group; p.H = d.heads;
    p.Hkv = d.kv_heads; p.rows = d.rows; p.max_steps = d.max_steps; p.ncols = d.beams * d.group; p.stages = stages;
    p.scale2 = 1.4426950408889634f / sqrtf((float)D);
    const unsigned grid = (unsigned)((size_t)d.batch * d.kv_heads * a.splits);
    kern<<<grid, 32 * (CW + 1), smem, st>>>(tmk, tmv, p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const Dims& d, const SdpaArgs& a, const CUtensorMap& tmk, const CUtensorMap& tmv, int stages,
                     cudaStream_t st) {
    const int nt = (d.beams * d.group + 7) / 8;
    if (nt == 1) {
        switch (d.head_dim) {
            case 64: return launch_one<T, 64, 1, 4>(d, a, tmk, tmv, stages, st);
            case 128: return launch_one<T, 128, 1, 4>(d, a, tmk, tmv, stages, st);
            case 256: return launch_one<T, 256, 1, 2>(d, a, tmk, tmv, stages, st);
        }
    } else if (nt == 2) {
        switch (d.head_dim) {
            case 64: return launch_one<T, 64, 2, 4>(d, a, tmk, tmv, stages, st);
            case 128: return launch_one<T, 128, 2, 4>(d, a, tmk, tmv, stages, st);
        }
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool tiled_supported(const Dims& d) {
    const int nt = (d.beams * d.group + 7) / 8;
    return nt == 1 || (nt == 2 && d.head_dim <= 128);
}

int tiled_tile_keys(int head_dim) { return head_dim == 256 ? 32 : 64; }

size_t tiled_smem_bytes(const Dims& d, int stages) {
    const int nt = (d.beams * d.group + 7) / 8;
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
