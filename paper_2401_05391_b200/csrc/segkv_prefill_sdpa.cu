// Prefill attention over the prompt segment (paper Section 3.1 / 3.3: the prefill kernel is
// the special case of the customised SDPA kernel that sees only the query and the prompt
// key/value, batch-first in and out): causal self-attention of every prompt position,
//     out[b,i,h,:] = softmax_{j<=i}( q[b,i,h,:] . K[b,j,:] / sqrt(D) + bias ) . V[b,j,:],
// with K/V read from the head-major prompt segment that segkv_prefill_write has just stored.
//
// Dense work, so it is laid out as a flash-attention forward: a CTA owns 128 query rows of one
// (request, head) (64 rows for head_dim 256), consumer warps take 16 rows each, a producer warp streams 64-key K/V
// tiles through a TMA-fed, 128-byte-swizzled shared-memory ring (the same tensor maps and tile
// layout as the decode kernel).  S = Q.K^T and O += P.V run on tensor cores (mma.sync
// m16n8k16, fp32 accumulate; Q fragments stay in registers, P is re-used as the A operand
// straight from the score accumulators), softmax is online in fp32 with base-2 exponents, and
// only the diagonal tile is masked.  Query tiles are issued longest first.
#include "segkv_internal.h"
#include "segkv_ptx.cuh"

namespace segkv_impl {

namespace {

using namespace ptx;

struct PrefillParams {
    const void* q;       // [B, N, H, D] token-major
    void* out;           // [B, N, H, D]
    const float* slopes; // [H] or NULL
    int* err_word;
    int N, H, Hkv, G, stages;
    float scale2;        // log2(e) / sqrt(D)
};

// Shape of one instantiation: kPW consumer warps (16 query rows each), kBN keys per K/V tile (the
// row count of the prompt segment's tensor-map box: 64, or 32 for head_dim 256), and whether Q
// stays in registers or, when it would not fit beside the O accumulators (head_dim 256), is
// staged once in shared memory and re-read with ldmatrix for every tile.
template <int D, int kPW, int kBN, bool QSMEM>
struct PrefillLayout {
    static constexpr int kBM = 16 * kPW;
    static constexpr int BOX_BYTES = kBN * 128;
    static constexpr int TILE_BYTES = kBN * D * 2;
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int Q_BYTES = QSMEM ? kBM * D * 2 : 0;
    static constexpr size_t bytes(int stages) {
        return 1024 + (size_t)stages * STAGE_BYTES + Q_BYTES + (size_t)stages * 16 + 64;
    }
};

template <typename T, int D, int kPW, int kBN, bool QSMEM>
__global__ void __launch_bounds__(32 * (kPW + 1), (kPW <= 4 && D <= 128) ? 2 : 1)
prefill_sdpa_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const PrefillParams p) {
    using L = PrefillLayout<D, kPW, kBN, QSMEM>;
    constexpr int kBM = L::kBM;
    constexpr int NT = kBN / 8;    // 8-key score column tiles per K/V tile
    constexpr int KS = D / 16;     // k-steps of Q.K^T
    constexpr int DT = D / 8;      // 8-wide output column tiles of O
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stages = p.stages;
    uint8_t* q_smem = smem + (size_t)stages * L::STAGE_BYTES;            // [kBM][D], 16-byte chunks XOR-swizzled by row
    uint64_t* bars = reinterpret_cast<uint64_t*>(q_smem + L::Q_BYTES);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + stages);
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;        // longest tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / p.G;
    const int nkt = min((p.N + kBN - 1) / kBN, ((qt + 1) * kBM + kBN - 1) / kBN);   // causal: tiles up to the CTA's last row

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kPW);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();

    if (warp == kPW) {
        // ------------------------------- producer warp -------------------------------
        if (lane == 0) {
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_v);
            bool ok = true;
            for (int kt = 0; kt < nkt && ok; ++kt) {
                const int st = kt % stages;
                ok = mbar_wait(empty0 + 8 * st, (((uint32_t)(kt / stages)) & 1) ^ 1);
                if (!ok) break;
                const uint32_t full = full0 + 8 * st;
                const uint32_t k_dst = smem_u32(smem + (size_t)st * L::STAGE_BYTES);
                const uint32_t v_dst = k_dst + L::TILE_BYTES;
                mbar_arrive_expect_tx(full, (uint32_t)L::STAGE_BYTES);
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx) {
                    tma_load_4d(k_dst + bx * L::BOX_BYTES, &tm_k, bx * 64, kvh, kt * kBN, b, full);
                    tma_load_4d(v_dst + bx * L::BOX_BYTES, &tm_v, bx * 64, kvh, kt * kBN, b, full);
                }
            }
            if (!ok) s_abort = 1;
        }
        return;
    }

    // --------------------------------- consumer warps ---------------------------------
    const int row0 = qt * kBM + warp * 16 + (lane >> 2);        // this lane's two query rows
    const int row1 = row0 + 8;
    const T* qbase = reinterpret_cast<const T*>(p.q) + ((size_t)b * p.N * p.H + h) * D;
    const size_t qstride = (size_t)p.H * D;                      // elements between tokens
    // Q as the A operand (a0/a2 from row0, a1/a3 from row1): resident in registers, or staged in
    // shared memory by all consumer warps (rows past the prompt as zeros) and fetched per k-step
    uint32_t qf[QSMEM ? 1 : KS][4];
    if constexpr (QSMEM) {
        constexpr int CPR = D / 8;                               // 16-byte chunks per row
        for (int i = tid; i < kBM * CPR; i += 32 * kPW) {
            const int r = i / CPR, c = i % CPR, grow = qt * kBM + r;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (grow < p.N) v = *reinterpret_cast<const uint4*>(qbase + (size_t)grow * qstride + c * 8);
            *reinterpret_cast<uint4*>(q_smem + (size_t)r * (D * 2) + (size_t)((c & ~7) | ((c ^ r) & 7)) * 16) = v;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kPW) : "memory");      // consumer warps only
    } else {
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int d0 = ks * 16 + (lane & 3) * 2;
            const uint32_t* r0 = reinterpret_cast<const uint32_t*>(qbase + (size_t)row0 * qstride + d0);
            const uint32_t* r1 = reinterpret_cast<const uint32_t*>(qbase + (size_t)row1 * qstride + d0);
            qf[ks][0] = row0 < p.N ? r0[0] : 0u;
            qf[ks][1] = row1 < p.N ? r1[0] : 0u;
            qf[ks][2] = row0 < p.N ? r0[4] : 0u;      // +8 elements
            qf[ks][3] = row1 < p.N ? r1[4] : 0u;
        }
    }
    // this lane's row address for ldmatrix of the staged Q: matrices (rows 0-7 | 8-15) x (k low | high)
    const int q_lrow = warp * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
    const float slope2 = p.slopes ? p.slopes[h] * 1.4426950408889634f : 0.f;

    float o_acc[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    bool ok = true;
    for (int kt = 0; kt < nkt; ++kt) {
        const int st = kt % stages;
        ok = mbar_wait(full0 + 8 * st, ((uint32_t)(kt / stages)) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t k_src = smem_u32(smem + (size_t)st * L::STAGE_BYTES);
        const uint32_t v_src = k_src + L::TILE_BYTES;
        const int wrow_lo = qt * kBM + warp * 16;                // this warp's rows: wrow_lo .. wrow_lo + 15
        if (kt * kBN > wrow_lo + 15) {                           // tile entirely above the diagonal for this warp
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * st);
            continue;
        }
        auto chunk_addr = [&](uint32_t base, int key, int ch) -> uint32_t {
            return base + (uint32_t)(ch >> 3) * L::BOX_BYTES + (uint32_t)key * 128 + (uint32_t)(((ch & 7) ^ (key & 7)) << 4);
        };
        // ---- S[16 rows, 64 keys] = Q . K^T ----
        float sc[NT][4];
#pragma unroll
        for (int i = 0; i < NT; ++i) sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
        {
            const int mi = lane >> 3;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t qa[4];
                if constexpr (QSMEM) {
                    const int c = 2 * ks + (lane >> 4);
                    ldmatrix_x4(qa, smem_u32(q_smem) + (uint32_t)q_lrow * (D * 2) +
                                        (uint32_t)((c & ~7) | ((c ^ q_lrow) & 7)) * 16);
                } else {
                    qa[0] = qf[ks][0]; qa[1] = qf[ks][1]; qa[2] = qf[ks][2]; qa[3] = qf[ks][3];
                }
#pragma unroll
                for (int nt2 = 0; nt2 < NT / 2; ++nt2) {
                    const int key = nt2 * 16 + (mi >> 1) * 8 + (lane & 7);
                    uint32_t bf[4];
                    ldmatrix_x4(bf, chunk_addr(k_src, key, 2 * ks + (mi & 1)));
                    Mma<T>::run(sc[2 * nt2], qa, bf[0], bf[1]);
                    Mma<T>::run(sc[2 * nt2 + 1], qa, bf[2], bf[3]);
                }
            }
        }
        // ---- scale, ALiBi, causal mask (diagonal tile only), online softmax ----
        const int key0 = kt * kBN + (lane & 3) * 2;              // key of sc[nt][0] is key0 + 8*nt
        const bool diag = kt * kBN + kBN - 1 > wrow_lo;          // some key of the tile is above some row of the warp
        float tmax[2] = {-INFINITY, -INFINITY};
        if (diag || p.slopes) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int key = key0 + 8 * nt + (i & 1);
                    const int row = (i & 2) ? row1 : row0;
                    float v = sc[nt][i] * p.scale2 + slope2 * (float)(key - row);
                    if (diag && key > row) v = -INFINITY;
                    sc[nt][i] = v;
                    tmax[i >> 1] = fmaxf(tmax[i >> 1], v);
                }
            }
        } else {                                                 // the common tile: scale only
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float v = sc[nt][i] * p.scale2;
                    sc[nt][i] = v;
                    tmax[i >> 1] = fmaxf(tmax[i >> 1], v);
                }
            }
        }
        float alpha[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float tm = tmax[r];
            tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 1));
            tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 2));
            const float m_new = fmaxf(m_run[r], tm);             // finite: key 0 is visible to every row
            alpha[r] = exp2f(m_run[r] - m_new);
            m_run[r] = m_new;
        }
        float lsum[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float e = exp2f(sc[nt][i] - m_run[i >> 1]);
                sc[nt][i] = e;
                lsum[i >> 1] += e;
            }
        }
        l_run[0] = l_run[0] * alpha[0] + lsum[0];
        l_run[1] = l_run[1] * alpha[1] + lsum[1];
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
            for (int dt = 0; dt < DT; ++dt) {
                o_acc[dt][0] *= alpha[0];
                o_acc[dt][1] *= alpha[0];
                o_acc[dt][2] *= alpha[1];
                o_acc[dt][3] *= alpha[1];
            }
        }
        // ---- O[16 rows, D] += P . V, P taken from the score accumulators as the A operand ----
        {
            const int mi = lane >> 3;
#pragma unroll
            for (int kk = 0; kk < NT / 2; ++kk) {
                uint32_t pa[4];
                pa[0] = Mma<T>::pack(sc[2 * kk][0], sc[2 * kk][1]);
                pa[1] = Mma<T>::pack(sc[2 * kk][2], sc[2 * kk][3]);
                pa[2] = Mma<T>::pack(sc[2 * kk + 1][0], sc[2 * kk + 1][1]);
                pa[3] = Mma<T>::pack(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
                const int key = kk * 16 + (mi & 1) * 8 + (lane & 7);
#pragma unroll
                for (int dn2 = 0; dn2 < D / 16; ++dn2) {
                    uint32_t bf[4];
                    ldmatrix_x4_trans(bf, chunk_addr(v_src, key, 2 * dn2 + (mi >> 1)));
                    Mma<T>::run(o_acc[2 * dn2], pa, bf[0], bf[1]);
                    Mma<T>::run(o_acc[2 * dn2 + 1], pa, bf[2], bf[3]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * st);
    }
    if (!ok) {
        if (lane == 0) atomicOr(p.err_word, SEGKV_DEV_WAIT_LIMIT);
        return;                                                  // output left untouched
    }

    // ---- normalise and store (token-major, like the input) ----
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float l = l_run[r];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        l_run[r] = 1.f / l;
    }
    T* obase = reinterpret_cast<T*>(p.out) + ((size_t)b * p.N * p.H + h) * D;
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) {
        const int d0 = dt * 8 + (lane & 3) * 2;
        if (row0 < p.N)
            *reinterpret_cast<uint32_t*>(obase + (size_t)row0 * qstride + d0) =
                Mma<T>::pack(o_acc[dt][0] * l_run[0], o_acc[dt][1] * l_run[0]);
        if (row1 < p.N)
            *reinterpret_cast<uint32_t*>(obase + (size_t)row1 * qstride + d0) =
                Mma<T>::pack(o_acc[dt][2] * l_run[1], o_acc[dt][3] * l_run[1]);
    }
}

template <typename T, int D, int kPW, int kBN, bool QSMEM>
cudaError_t launch_prefill(const Dims& d, const PrefillArgs& a, cudaStream_t st) {
    using L = PrefillLayout<D, kPW, kBN, QSMEM>;
    const int stages = D <= 64 ? 4 : 3;
    const size_t smem = L::bytes(stages);
    auto kern = prefill_sdpa_kernel<T, D, kPW, kBN, QSMEM>;
    static bool configured[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    PrefillParams p;
    p.q = a.q; p.out = a.out; p.slopes = a.slopes; p.err_word = a.err_word;
    p.N = a.prompt_len; p.H = d.heads; p.Hkv = d.kv_heads; p.G = d.group; p.stages = stages;
    p.scale2 = 1.4426950408889634f / sqrtf((float)D);
    dim3 grid((unsigned)((a.prompt_len + L::kBM - 1) / L::kBM), (unsigned)d.heads, (unsigned)d.batch);
    kern<<<grid, 32 * (kPW + 1), smem, st>>>(*a.tm_k, *a.tm_v, p);
    return cudaGetLastError();
}

}  // namespace

bool prefill_sdpa_supported(const Dims& d) { return d.head_dim == 64 || d.head_dim == 128 || d.head_dim == 256; }

cudaError_t launch_prefill_sdpa(const Dims& d, const PrefillArgs& a, cudaStream_t st) {
    if (prefill_tc5_supported(d)) return launch_prefill_tc5(d, a, st);
    const bool bf = d.dtype == SEGKV_BF16;
    switch (d.head_dim) {
        case 64:
            return bf ? launch_prefill<__nv_bfloat16, 64, 4, 64, false>(d, a, st)
                      : launch_prefill<__half, 64, 4, 64, false>(d, a, st);
        case 128:
            return bf ? launch_prefill<__nv_bfloat16, 128, 4, 64, false>(d, a, st)
                      : launch_prefill<__half, 128, 4, 64, false>(d, a, st);
        case 256:   // 32-key tiles (the prompt segment's box for this head size), Q staged in shared memory
            return bf ? launch_prefill<__nv_bfloat16, 256, 4, 32, true>(d, a, st)
                      : launch_prefill<__half, 256, 4, 32, true>(d, a, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace segkv_impl
