// Prefill attention on the fifth-generation tensor cores (tcgen05 + tensor memory), head_dim 128.
//
// Same operation as segkv_prefill_sdpa.cu (paper Section 3.1 / 3.3: causal attention of the
// prompt, batch-first in and out, K/V from the prompt segment), laid out for tcgen05:
//
//   * a CTA owns 128 query rows of one (request, head): one row per TMEM lane;
//   * Q [128 x 128] is staged once in shared memory in the 128-byte-swizzled K-major layout,
//     K/V tiles of 64 keys arrive by TMA in the same layout (the prompt segment's tensor maps);
//   * one elected thread issues the MMAs: S = Q.K^T (M 128, N 64, eight K-steps of 16) into one
//     of two 64-column TMEM buffers, and O += P.V (M 128, N 128, four K-steps) into a 128-column
//     TMEM accumulator; V is consumed as an MN-major B operand straight from its row-major tile;
//   * four softmax warps own one row per thread: they read S with tcgen05.ld (no shuffles for
//     the row max / sum), write P as bf16/fp16 into a swizzled shared-memory tile that the next
//     MMA takes as its A operand, and rescale O in tensor memory only when a row's maximum has
//     grown by more than 2^8 since the reference it is using (the sum uses the same reference,
//     so the result is exact);
//   * S is double-buffered, so Q.K^T of tile j+1 runs under the softmax of tile j and P.V of
//     tile j under the softmax of tile j+1.
//
// Every mbarrier wait is bounded; on expiry the kernel flags SEGKV_DEV_WAIT_LIMIT, skips the
// output and still releases its tensor memory.
#include "segkv_internal.h"
#include "segkv_ptx.cuh"

namespace segkv_impl {

namespace {

using namespace ptx;

constexpr int kD = 128;        // head_dim of this kernel
constexpr int kRows = 128;     // query rows per CTA (TMEM lanes)
constexpr int kKeys = 64;      // keys per K/V tile
constexpr int kStages = 3;
constexpr int kBoxKV = kKeys * 128;          // one 64-element-wide box of a K/V tile
constexpr int kTileKV = kKeys * kD * 2;      // bytes of a K (or V) tile
constexpr int kBoxQ = kRows * 128;           // one box of the Q tile
constexpr int kTmemCols = 256;               // S0 [0,64)  S1 [64,128)  O [128,256)

struct Tc5Params {
    const void* q;
    void* out;
    const float* slopes;
    int* err_word;
    int N, H, Hkv, G;
    float scale2;
    uint32_t idesc_qk, idesc_pv;
};

// shared memory: | K/V ring (kStages x 32 KB) | Q 32 KB | P 16 KB | barriers | tmem slot |
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * 2 * kTileKV + 2 * kBoxQ + kBoxQ + 256;

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// 32 lanes x 32 columns of 32-bit words: this thread's TMEM lane, 32 consecutive columns
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
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

template <typename T>
__global__ void __launch_bounds__(192, 1)
prefill_tc5_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const Tc5Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* q_smem = smem + (size_t)kStages * 2 * kTileKV;      // two boxes [128 rows][64 elements], swizzled
    uint8_t* p_smem = q_smem + 2 * kBoxQ;                         // one box [128 rows][64 keys], swizzled
    uint64_t* bars = reinterpret_cast<uint64_t*>(p_smem + kBoxQ);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kStages);
    const uint32_t bar_s0 = smem_u32(bars + 2 * kStages);         // two: S buffer written
    const uint32_t bar_p = bar_s0 + 16;                           // P tile written, S buffer read
    const uint32_t bar_o = bar_s0 + 24;                           // P.V of a tile complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;          // longest tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int slab = b * p.Hkv + h / p.G;
    const int nkt = min((p.N + kKeys - 1) / kKeys, ((qt + 1) * kRows + kKeys - 1) / kKeys);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(bar_s0, 1);
        mbar_init(bar_s0 + 8, 1);
        mbar_init(bar_p, 128);
        mbar_init(bar_o, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 5) {                                              // this warp owns the tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // stage Q (rows past the prompt as zeros): element (r, d) -> box d/64, row r, 16-byte chunk
    // ((d%64)/8) ^ (r%8): the layout TMA's 128-byte swizzle would have produced
    const T* qbase = reinterpret_cast<const T*>(p.q) + ((size_t)b * p.N * p.H + h) * kD;
    const size_t qstride = (size_t)p.H * kD;
    for (int i = tid; i < kRows * 16; i += 192) {
        const int r = i >> 4, c = i & 15, grow = qt * kRows + r;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (grow < p.N) v = *reinterpret_cast<const uint4*>(qbase + (size_t)grow * qstride + c * 8);
        *reinterpret_cast<uint4*>(q_smem + (size_t)(c >> 3) * kBoxQ + (size_t)r * 128 + (size_t)(((c ^ r) & 7) << 4)) = v;
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tm_o = tmem + 128;                             // O accumulator columns

    if (warp == 4) {
        // ------------------------------- TMA producer -------------------------------
        if (lane == 0) {
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_v);
            for (int kt = 0; kt < nkt; ++kt) {
                const int st = kt % kStages;
                if (!mbar_wait(empty0 + 8 * st, (((uint32_t)(kt / kStages)) & 1) ^ 1)) { s_abort = 1; break; }
                const uint32_t full = full0 + 8 * st;
                const uint32_t k_dst = smem_u32(smem + (size_t)st * 2 * kTileKV);
                const uint32_t v_dst = k_dst + kTileKV;
                mbar_arrive_expect_tx(full, 2u * kTileKV);
#pragma unroll
                for (int bx = 0; bx < 2; ++bx) {
                    tma_load_3d(k_dst + bx * kBoxKV, &tm_k, bx * 64, kt * kKeys, slab, full);
                    tma_load_3d(v_dst + bx * kBoxKV, &tm_v, bx * 64, kt * kKeys, slab, full);
                }
            }
        }
    } else if (warp == 5) {
        // -------------------------------- MMA issuer --------------------------------
        if (lane == 0) {
            const uint32_t q_addr = smem_u32(q_smem), p_addr = smem_u32(p_smem);
            auto issue_qk = [&](int kt) -> bool {                 // S[kt & 1] = Q . K_kt^T
                const int st = kt % kStages;
                if (!mbar_wait(full0 + 8 * st, ((uint32_t)(kt / kStages)) & 1)) return false;
                tc_fence_after();
                const uint32_t k_addr = smem_u32(smem + (size_t)st * 2 * kTileKV);
#pragma unroll
                for (int ks = 0; ks < kD / 16; ++ks) {
                    const uint32_t off = (uint32_t)(ks & 3) * 32;
                    tc_mma(tmem + (uint32_t)(kt & 1) * 64,
                           smem_desc(q_addr + (ks >> 2) * kBoxQ + off, 16, 1024),
                           smem_desc(k_addr + (ks >> 2) * kBoxKV + off, 16, 1024), p.idesc_qk, ks > 0);
                }
                tc_commit(bar_s0 + 8 * (kt & 1));
                return true;
            };
            bool ok = issue_qk(0);
            for (int kt = 0; kt < nkt && ok; ++kt) {
                if (kt + 1 < nkt) ok = issue_qk(kt + 1);          // runs under the softmax of tile kt
                if (!ok) break;
                ok = mbar_wait(bar_p, (uint32_t)kt & 1);
                if (!ok) break;
                tc_fence_after();
                const int st = kt % kStages;
                const uint32_t v_addr = smem_u32(smem + (size_t)st * 2 * kTileKV) + kTileKV;
#pragma unroll
                for (int kk = 0; kk < kKeys / 16; ++kk)           // O += P[:, 16 keys] . V[16 keys, :]
                    tc_mma(tm_o, smem_desc(p_addr + kk * 32, 16, 1024),
                           smem_desc(v_addr + kk * 2048, kBoxKV, 1024), p.idesc_pv, (kt > 0 || kk > 0));
                tc_commit(empty0 + 8 * st);                       // K/V stage free once these MMAs are done
                tc_commit(bar_o);
            }
            if (!ok) s_abort = 1;
        }
    } else {
        // ------------------------------ softmax warps: one row per thread ------------------------------
        const int row = qt * kRows + tid;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;    // this warp's TMEM lanes
        const float slope2 = p.slopes ? p.slopes[h] * 1.4426950408889634f : 0.f;
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int kt = 0; kt < nkt; ++kt) {
            ok = mbar_wait(bar_s0 + 8 * (kt & 1), ((uint32_t)(kt >> 1)) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t sr[2][32];
            tc_ld32(tmem + lane_base + (uint32_t)(kt & 1) * 64, sr[0]);
            tc_ld32(tmem + lane_base + (uint32_t)(kt & 1) * 64 + 32, sr[1]);
            tc_wait_ld();
            const int key0 = kt * kKeys;
            const bool diag = key0 + kKeys - 1 > qt * kRows;       // some key above some row of the CTA
            float tmax = -INFINITY;
            float* sv = reinterpret_cast<float*>(&sr[0][0]);
            if (diag || p.slopes) {
#pragma unroll
                for (int i = 0; i < kKeys; ++i) {
                    const int key = key0 + i;
                    float v = sv[i] * p.scale2 + slope2 * (float)(key - row);
                    if (diag && key > row) v = -INFINITY;
                    sv[i] = v;
                    tmax = fmaxf(tmax, v);
                }
            } else {
#pragma unroll
                for (int i = 0; i < kKeys; ++i) {
                    sv[i] *= p.scale2;
                    tmax = fmaxf(tmax, sv[i]);
                }
            }
            // a new reference only when the maximum has grown by more than 2^8: exponentials stay
            // below 2^8 of the reference, the sum and O use the same reference
            const bool need = tmax > m_ref + 8.f;
            float alpha = 1.f;
            if (need) {
                alpha = exp2f(m_ref - tmax);                       // 0 on the first tile
                m_ref = tmax;
            }
            float lsum = 0.f;
            uint32_t pk[kKeys / 2];
#pragma unroll
            for (int i = 0; i < kKeys; i += 2) {
                const float e0 = exp2f(sv[i] - m_ref), e1 = exp2f(sv[i + 1] - m_ref);
                lsum += e0 + e1;
                pk[i >> 1] = Mma<T>::pack(e0, e1);
            }
            l_run = l_run * alpha + lsum;
            if (kt > 0) {
                ok = mbar_wait(bar_o, (uint32_t)(kt - 1) & 1);     // P.V of the previous tile done: P free, O stable
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                if (__any_sync(0xffffffffu, need)) {
#pragma unroll
                    for (int c = 0; c < kD / 32; ++c) {
                        uint32_t orr[32];
                        tc_ld32(tm_o + lane_base + c * 32, orr);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
                        tc_st32(tm_o + lane_base + c * 32, orr);
                    }
                    tc_wait_st();
                }
            }
            // P row -> shared memory, K-major with the 128-byte swizzle (eight 16-byte chunks)
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(p_smem + (size_t)tid * 128 + (size_t)(((c ^ tid) & 7) << 4)) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar_p);
        }
        if (ok) {
            ok = mbar_wait(bar_o, (uint32_t)(nkt - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l_run;
            T* orow = reinterpret_cast<T*>(p.out) + ((size_t)b * p.N * p.H + h) * kD + (size_t)row * qstride;
#pragma unroll
            for (int c = 0; c < kD / 32; ++c) {
                uint32_t orr[32];
                tc_ld32(tm_o + lane_base + c * 32, orr);
                tc_wait_ld();
                if (row < p.N) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        *reinterpret_cast<uint4*>(orow + c * 32 + i * 8) = make_uint4(
                            Mma<T>::pack(__uint_as_float(orr[8 * i]) * inv, __uint_as_float(orr[8 * i + 1]) * inv),
                            Mma<T>::pack(__uint_as_float(orr[8 * i + 2]) * inv, __uint_as_float(orr[8 * i + 3]) * inv),
                            Mma<T>::pack(__uint_as_float(orr[8 * i + 4]) * inv, __uint_as_float(orr[8 * i + 5]) * inv),
                            Mma<T>::pack(__uint_as_float(orr[8 * i + 6]) * inv, __uint_as_float(orr[8 * i + 7]) * inv));
                }
            }
        } else if (lane == 0) {
            s_abort = 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
        if (lane == 0 && s_abort) atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
    }
}

}  // namespace

bool prefill_tc5_supported(const Dims& d) { return d.head_dim == kD; }

cudaError_t launch_prefill_tc5(const Dims& d, const PrefillArgs& a, cudaStream_t st) {
    if (d.head_dim != kD) return cudaErrorInvalidValue;
    const bool bf = d.dtype == SEGKV_BF16;
    static bool configured[64][2] = {{false}};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev][bf]) {
        cudaError_t e = bf ? cudaFuncSetAttribute(prefill_tc5_kernel<__nv_bfloat16>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes)
                           : cudaFuncSetAttribute(prefill_tc5_kernel<__half>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev][bf] = true;
    }
    Tc5Params p;
    p.q = a.q; p.out = a.out; p.slopes = a.slopes; p.err_word = a.err_word;
    p.N = a.prompt_len; p.H = d.heads; p.Hkv = d.kv_heads; p.G = d.group;
    p.scale2 = 1.4426950408889634f / sqrtf((float)kD);
    // instruction descriptor: fp32 accumulate, A/B format, operand majors, N >> 3, M >> 4
    const uint32_t fmt = bf ? 1u : 0u;
    const uint32_t common = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kRows >> 4) << 24);
    p.idesc_qk = common | ((uint32_t)(kKeys >> 3) << 17);                 // A, B both K-major
    p.idesc_pv = common | (1u << 16) | ((uint32_t)(kD >> 3) << 17);       // B (= V) MN-major
    dim3 grid((unsigned)((a.prompt_len + kRows - 1) / kRows), (unsigned)d.heads, (unsigned)d.batch);
    if (bf) prefill_tc5_kernel<__nv_bfloat16><<<grid, 192, kSmemBytes, st>>>(*a.tm_k, *a.tm_v, p);
    else prefill_tc5_kernel<__half><<<grid, 192, kSmemBytes, st>>>(*a.tm_k, *a.tm_v, p);
    return cudaGetLastError();
}

}  // namespace segkv_impl
