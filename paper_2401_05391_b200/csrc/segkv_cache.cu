// Cache-maintenance kernels: prompt store at prefill, per-step append and the
// beam-index (ancestry) update.
#include "segkv_internal.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace segkv_impl {

// ---------------------------------------------------------------------------
// Prompt store (paper Section 3.2: prompt K/V generated at prefill and kept
// once per request).  Input token-major [B, P, Hkv, D]; stored head-major
// [B, Hkv, max_prompt, D] so that each (request, kv head) slab is one
// contiguous [P, D] matrix the attention kernel can fetch with 2-D TMA boxes.
// One thread moves one 16-byte chunk; consecutive threads read consecutive
// chunks of the source.
// ---------------------------------------------------------------------------
__global__ void prefill_transpose_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v,
                                         uint4* __restrict__ kp, uint4* __restrict__ vp, int B, int P,
                                         int Hkv, int chunks /* D*2/16 */, long long sb, long long sh,
                                         long long sp /* strides in 16-byte chunks */,
                                         const int32_t* __restrict__ plens) {
    const long long total = (long long)B * P * Hkv * chunks;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int c = (int)(i % chunks);
        long long r = i / chunks;
        int h = (int)(r % Hkv);
        r /= Hkv;
        int p = (int)(r % P);
        int b = (int)(r / P);
        long long dst = b * sb + h * sh + p * sp + c;
        // ragged prompts: the padding of a shorter request is stored as zeros, so that a masked
        // key can never put a NaN or an infinity into a weighted sum
        const bool pad = plens && p >= plens[b];
        kp[dst] = pad ? make_uint4(0u, 0u, 0u, 0u) : k[i];
        vp[dst] = pad ? make_uint4(0u, 0u, 0u, 0u) : v[i];
    }
}

cudaError_t launch_prefill_transpose(const Dims& d, const void* k, const void* v, void* kp, void* vp, const int32_t* plens,
                                     int prompt_len, int sm_count, cudaStream_t st) {
    const int chunks = d.head_dim * 2 / 16;
    const PromptStrides ps = prompt_strides(d);
    long long total = (long long)d.batch * prompt_len * d.kv_heads * chunks;
    if (total == 0) return cudaSuccess;
    int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > (long long)sm_count * 32) blocks = (long long)sm_count * 32;
    prefill_transpose_kernel<<<(unsigned)blocks, threads, 0, st>>>(
        (const uint4*)k, (const uint4*)v, (uint4*)kp, (uint4*)vp, d.batch, prompt_len, d.kv_heads, chunks,
        ps.b / 8, ps.h / 8, ps.p / 8, plens);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Append + beam-index update, one launch per decode step.
//
// Blocks [0, B) update the beam-index table of one request each; the remaining
// blocks copy the step's new K/V rows into slab `step` of the response segment
// (Section 3.1: Key_t / Value_t are kept in place, no Cat) and record the
// parent ids as row `step` of the parent table.
//
// Index table (Section 3.3, "Index select fusion"): anc_t[g][s] is the row of
// slab s that beam slot g reads.  Re-ordering the whole past cache by the beam
// indices at every step (Section 3.1) is the recurrence
//     anc_t[g][s] = anc_{t-1}[ b*W + parent_t[g] ][s]   for s < t,
//     anc_t[g][t] = g,
// which is independent per s, so one thread takes one step s and the update
// has no serial chain.  Two generations are kept (t & 1).
//
// While the W rows of a step are in registers the same thread also emits the
// step's DISTINCT rows with the set of beams that read each (a bit mask), and
// a block-wide prefix sum packs them into the request's list.  The attention
// kernel walks that list, so a row shared by several beams is fetched once.
// ---------------------------------------------------------------------------
constexpr int kBtThreads = 256;

__device__ __forceinline__ int warp_incl_scan(int v) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, v, o);
        if ((threadIdx.x & 31) >= o) v += n;
    }
    return v;
}

// Eight 16-bit values of one 16-byte chunk <-> fp32.
__device__ __forceinline__ void unpack8(const uint4& v, bool bf16, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (bf16) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        } else {
            const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
}
__device__ __forceinline__ uint4 pack8(const float* f, bool bf16) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (bf16) {
            const __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&t);
        } else {
            const __half2 t = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&t);
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// The copy blocks' K rows with the rotary embedding applied on the way (fp32 arithmetic, one
// rounding): pair i of a row is (x[i], x[i + D/2]) (half-split) or (x[2i], x[2i+1])
// (interleaved) and turns by the angle whose cos / sin the tables hold for the row's position.
__device__ __forceinline__ void rope_copy(const RopeArgs& r, int W, int step, const uint4* __restrict__ k_new,
                                          const uint4* __restrict__ v_new, uint4* __restrict__ kr_slab,
                                          uint4* __restrict__ vr_slab, long long slab_chunks, long long first,
                                          long long stride) {
    const int cpr = r.head_dim / 8;                               // 16-byte chunks per (row, head)
    const int half_d = r.head_dim / 2;
    if (r.style == SEGKV_ROPE_INTERLEAVED) {
        for (long long i = first; i < slab_chunks; i += stride) {
            const int c = (int)(i % cpr);
            const int b = (int)(i / cpr / r.kv_heads) / W;
            const int pos = (r.plens ? r.plens[b] : r.prompt_len) + step;
            const float* cs = r.cos + (size_t)pos * half_d + c * 4;
            const float* sn = r.sin + (size_t)pos * half_d + c * 4;
            float x[8];
            unpack8(k_new[i], r.bf16, x);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float a = x[2 * e], bb = x[2 * e + 1];
                x[2 * e] = a * cs[e] - bb * sn[e];
                x[2 * e + 1] = bb * cs[e] + a * sn[e];
            }
            kr_slab[i] = pack8(x, r.bf16);
            vr_slab[i] = v_new[i];
        }
    } else {
        const int hc = cpr / 2;                                   // chunks of the low half of a row
        for (long long j = first; j < slab_chunks / 2; j += stride) {
            const int c = (int)(j % hc);
            const long long rh = j / hc;                          // (row, head)
            const int b = (int)(rh / r.kv_heads) / W;
            const int pos = (r.plens ? r.plens[b] : r.prompt_len) + step;
            const float* cs = r.cos + (size_t)pos * half_d + c * 8;
            const float* sn = r.sin + (size_t)pos * half_d + c * 8;
            const long long lo = rh * cpr + c, hi = lo + hc;
            float xl[8], xh[8];
            unpack8(k_new[lo], r.bf16, xl);
            unpack8(k_new[hi], r.bf16, xh);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float a = xl[e], bb = xh[e];
                xl[e] = a * cs[e] - bb * sn[e];
                xh[e] = bb * cs[e] + a * sn[e];
            }
            kr_slab[lo] = pack8(xl, r.bf16);
            kr_slab[hi] = pack8(xh, r.bf16);
            vr_slab[lo] = v_new[lo];
            vr_slab[hi] = v_new[hi];
        }
    }
}

__global__ void __launch_bounds__(kBtThreads)
append_kernel(int B, int W, int rows, int max_steps, int step, const int32_t* __restrict__ beam_parent,
              const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* __restrict__ kr_slab,
              uint4* __restrict__ vr_slab, long long slab_chunks, int32_t* __restrict__ parent_row,
              const int32_t* __restrict__ anc_prev, int32_t* __restrict__ anc_cur, URow* __restrict__ ulist,
              int32_t* __restrict__ ucount, int* __restrict__ err_word, int rebuild, const RopeArgs rope) {
    // Programmatic dependent launch: this kernel touches nothing until the previous kernel of
    // the stream has completed, and only then lets the next one start its prologue (so a kernel
    // that starts early always finds everything older than its predecessor complete).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if ((int)blockIdx.x >= B) {
        // ---- copy blocks -------------------------------------------------
        const long long nb = gridDim.x - B;
        const long long first = ((long long)blockIdx.x - B) * blockDim.x + threadIdx.x;
        if (rope.style != 0) {
            rope_copy(rope, W, step, k_new, v_new, kr_slab, vr_slab, slab_chunks, first, nb * blockDim.x);
        } else {
            for (long long i = first; i < slab_chunks; i += nb * blockDim.x) {
                kr_slab[i] = k_new[i];
                vr_slab[i] = v_new[i];
            }
        }
        if (parent_row == nullptr) return;                     // K/V rows only: the tables belong to another handle
        if (beam_parent != nullptr)
            for (long long i = first; i < rows; i += nb * blockDim.x) parent_row[i] = beam_parent[i];
        else
            for (long long i = first; i < rows; i += nb * blockDim.x) parent_row[i] = (int)(i % W);
        return;
    }

    // ---- index-table block of request b ------------------------------------
    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    __shared__ int s_par[kMaxCols];
    __shared__ int s_warp[kBtThreads / 32];
    __shared__ int s_base;
    if (tid < W) {
        int p = tid;
        if (step > 0 && !rebuild) {
            p = beam_parent[b * W + tid];
            if (p < 0 || p >= W) {
                atomicOr(err_word, SEGKV_DEV_BAD_PARENT);
                p = p < 0 ? 0 : W - 1;
            }
        }
        s_par[tid] = p;
    }
    if (tid == 0) s_base = 0;
    __syncthreads();

    URow* list = ulist + (size_t)b * W * max_steps;
    const int n = step + 1;
    for (int s0 = 0; s0 < n; s0 += kBtThreads) {
        const int s = s0 + tid;
        int r[kMaxCols];
        int cnt = 0;
        if (s < n) {
#pragma unroll 4
            for (int j = 0; j < W; ++j) {
                int v;
                if (rebuild) {
                    v = anc_cur[(size_t)(b * W + j) * max_steps + s];    // the table is already this step's
                } else {
                    v = (s == step) ? b * W + j : anc_prev[(size_t)(b * W + s_par[j]) * max_steps + s];
                    anc_cur[(size_t)(b * W + j) * max_steps + s] = v;
                }
                r[j] = v;
            }
            for (int j = 0; j < W; ++j) {
                bool first = true;
                for (int i = 0; i < j; ++i) first = first && (r[i] != r[j]);
                cnt += first ? 1 : 0;
            }
        }
        // exclusive prefix of cnt over the block
        int incl = warp_incl_scan(cnt);
        if ((tid & 31) == 31) s_warp[tid >> 5] = incl;
        __syncthreads();
        int woff = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kBtThreads / 32; ++w) {
            int v = s_warp[w];
            if (w < (tid >> 5)) woff += v;
            total += v;
        }
        int pos = s_base + woff + incl - cnt;
        if (s < n) {
            for (int j = 0; j < W; ++j) {
                bool first = true;
                uint32_t mask = 0;
                for (int i = 0; i < W; ++i) {
                    bool same = (r[i] == r[j]);
                    if (same && i < j) first = false;
                    mask |= same ? (1u << i) : 0u;
                }
                if (first) {
                    URow u;
                    u.row = s * rows + r[j];
                    u.mask = mask;
                    list[pos++] = u;
                }
            }
        }
        __syncthreads();
        if (tid == 0) s_base += total;
        __syncthreads();
    }
    if (tid == 0) ucount[b] = s_base;
}

cudaError_t launch_append(const Dims& d, int step, const int32_t* beam_parent, const void* k_new,
                          const void* v_new, void* kr_slab_v, void* vr_slab_v, int32_t* parent_tab,
                          const int32_t* anc_prev, int32_t* anc_cur, URow* ulist, int32_t* ucount,
                          int* err_word, int sm_count, bool pdl, cudaStream_t st, const RopeArgs* rope, bool tables) {
    const long long slab_elems = (long long)d.rows * d.kv_heads * d.head_dim;
    const long long slab_chunks = slab_elems * 2 / 16;
    long long copy_blocks = (slab_chunks + kBtThreads * 4 - 1) / (kBtThreads * 4);
    if (copy_blocks < 1) copy_blocks = 1;
    if (copy_blocks > (long long)sm_count * 8) copy_blocks = (long long)sm_count * 8;
    uint4* kr_slab = (uint4*)kr_slab_v;     // slab of this step inside the response segment
    uint4* vr_slab = (uint4*)vr_slab_v;
    cudaLaunchConfig_t cfg = {};
    const int table_blocks = tables ? d.batch : 0;           // without tables every block copies rows
    cfg.gridDim = dim3((unsigned)(table_blocks + copy_blocks), 1, 1);
    cfg.blockDim = dim3(kBtThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (pdl) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    const int32_t* bp = step > 0 ? beam_parent : nullptr;
    return cudaLaunchKernelEx(&cfg, append_kernel, table_blocks, d.beams, d.rows, d.max_steps, step, bp,
                              (const uint4*)k_new, (const uint4*)v_new, kr_slab, vr_slab, slab_chunks,
                              tables ? parent_tab + (size_t)step * d.rows : (int32_t*)nullptr, anc_prev, anc_cur, ulist,
                              ucount, err_word, 0,
                              rope ? *rope : RopeArgs{});
}

// The distinct-row lists of the newest step from its beam-index table alone: the table blocks of
// the append kernel in read-only mode (used after fused decode steps, which skip the lists).
cudaError_t launch_rebuild_lists(const Dims& d, int steps, const int32_t* anc_cur, URow* ulist, int32_t* ucount,
                                 cudaStream_t st) {
    if (steps <= 0) return cudaSuccess;
    append_kernel<<<(unsigned)d.batch, kBtThreads, 0, st>>>(
        d.batch, d.beams, d.rows, d.max_steps, steps - 1, nullptr, nullptr, nullptr, nullptr, nullptr, 0, nullptr,
        nullptr, const_cast<int32_t*>(anc_cur), ulist, ucount, nullptr, 1, RopeArgs{});
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// A read-only stream over a buffer (16-byte loads folded into one word per thread, one word
// per block written): the bandwidth a kernel that only READS can reach on this GPU, which is what
// the decode attention does.  A copy's figure counts bytes read plus bytes written and sits lower.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) read_stream_kernel(const uint4* __restrict__ src, size_t n16,
                                                          unsigned* __restrict__ sink) {
    unsigned acc = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x * 4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x * 4 + threadIdx.x; i < n16; i += stride) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t k = i + (size_t)u * blockDim.x;
            v[u] = k < n16 ? __ldcs(src + k) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    acc ^= __shfl_xor_sync(0xffffffffu, acc, 16);
    acc ^= __shfl_xor_sync(0xffffffffu, acc, 8);
    acc ^= __shfl_xor_sync(0xffffffffu, acc, 4);
    acc ^= __shfl_xor_sync(0xffffffffu, acc, 2);
    acc ^= __shfl_xor_sync(0xffffffffu, acc, 1);
    if ((threadIdx.x & 31) == 0) atomicXor(sink + (blockIdx.x & 63), acc);
}

cudaError_t launch_read_stream(const void* src, size_t bytes, unsigned* sink, int sm_count, cudaStream_t st) {
    read_stream_kernel<<<(unsigned)(sm_count * 8), 256, 0, st>>>((const uint4*)src, bytes / 16, sink);
    return cudaGetLastError();
}

}  // namespace segkv_impl
