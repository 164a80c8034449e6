// Row-wise decode attention: one CTA per (beam slot, head), every beam reads its
// own rows through the beam-index table, fp32 ALU arithmetic.  This is the
// direct transcription of the paper's per-beam formulation (Section 3.3): loop
// over the prompt rows, then over the index-selected response rows, one online
// softmax across both.  It re-reads the prompt once per beam, so it is not the
// fast path; the library uses it for shapes the tiled kernel does not take and
// exposes it as a cross-check.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "segkv_internal.h"

namespace segkv_impl {

namespace {

template <typename T> struct Cvt;
template <> struct Cvt<__half> {
    static __device__ __forceinline__ float2 up(uint32_t u) {
        return __half22float2(*reinterpret_cast<const __half2*>(&u));
    }
    static __device__ __forceinline__ __half down(float f) { return __float2half_rn(f); }
};
template <> struct Cvt<__nv_bfloat16> {
    static __device__ __forceinline__ float2 up(uint32_t u) {
        return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u));
    }
    static __device__ __forceinline__ __nv_bfloat16 down(float f) { return __float2bfloat16_rn(f); }
};

template <int E> struct Vec;                       // E 16-bit elements as 32-bit words
template <> struct Vec<2> { using type = uint32_t; };
template <> struct Vec<4> { using type = uint2; };
template <> struct Vec<8> { using type = uint4; };

template <typename T, int E>
__device__ __forceinline__ void load_row(const T* p, float (&f)[E]) {
    typename Vec<E>::type raw = *reinterpret_cast<const typename Vec<E>::type*>(p);
    const uint32_t* w = reinterpret_cast<const uint32_t*>(&raw);
#pragma unroll
    for (int i = 0; i < E / 2; ++i) {
        float2 t = Cvt<T>::up(w[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

constexpr int kWarps = 4;

template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32)
sdpa_rowwise_kernel(const T* __restrict__ q, T* __restrict__ out, const float* __restrict__ slopes,
                    const T* __restrict__ kp, const T* __restrict__ vp, const T* __restrict__ kr,
                    const T* const* __restrict__ k_chunks, int chunk_steps, long long vdelta_elems,
                    const int32_t* __restrict__ anc, const int32_t* __restrict__ plens, int P_all, int steps, int W, int H,
                    int Hkv, int group, PromptStrides ps, int max_steps, int rows) {
    constexpr int E = D / 32;
    const int h = blockIdx.x, g = blockIdx.y;
    const int b = g / W, kvh = h / group;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    float qf[E];
    load_row<T, E>(q + ((size_t)g * H + h) * D + lane * E, qf);
    const float kLog2e = 1.4426950408889634f;
    const float scale2 = kLog2e / sqrtf((float)D);
    const float slope2 = slopes ? slopes[h] * kLog2e : 0.f;
    const int P = plens ? plens[b] : P_all;
    const int L = P + steps;
    const int qpos = L - 1;

    float m = -INFINITY, l = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;

    for (int i = warp; i < L; i += kWarps) {
        const T* krow;
        const T* vrow;
        if (i < P) {
            const size_t off = (size_t)(b * ps.b + kvh * ps.h + i * ps.p);
            krow = kp + off;
            vrow = vp + off;
        } else {
            const int s = i - P;
            const int r = anc[(size_t)g * max_steps + s];
            const size_t slab = (size_t)rows * Hkv * D;          // elements of one step
            const T* base = kr + (size_t)s * slab;                // one array, or the chunk that holds step s
            if (chunk_steps) base = k_chunks[s / chunk_steps] + (size_t)(s % chunk_steps) * slab;
            krow = base + ((size_t)r * Hkv + kvh) * D;
            vrow = krow + vdelta_elems;                           // V rows sit a constant behind their K rows
        }
        float kf[E], vf[E];
        load_row<T, E>(krow + lane * E, kf);
        load_row<T, E>(vrow + lane * E, vf);
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        float s2 = dot * scale2 + slope2 * (float)(i - qpos);
        float mn = fmaxf(m, s2);
        float alpha = exp2f(m - mn);
        float p = exp2f(s2 - mn);
        l = l * alpha + p;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = acc[e] * alpha + p * vf[e];
        m = mn;
    }

    __shared__ float s_m[kWarps], s_l[kWarps];
    __shared__ float s_acc[kWarps][D];
    if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < E; ++e) s_acc[warp][lane * E + e] = acc[e];
    __syncthreads();
    for (int d = threadIdx.x; d < D; d += kWarps * 32) {
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, s_m[w]);
        float ll = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            float f = (s_m[w] == -INFINITY) ? 0.f : exp2f(s_m[w] - mm);
            ll += s_l[w] * f;
            o += s_acc[w][d] * f;
        }
        out[((size_t)g * H + h) * D + d] = Cvt<T>::down(o / ll);
    }
}

template <typename T>
cudaError_t dispatch(const Dims& d, const SdpaArgs& a, cudaStream_t st) {
    dim3 grid(d.heads, d.rows), block(kWarps * 32);
#define SEGKV_ROWWISE(DD)                                                                               \
    sdpa_rowwise_kernel<T, DD><<<grid, block, 0, st>>>(                                                 \
        (const T*)a.q, (T*)a.out, a.slopes, (const T*)a.kp, (const T*)a.vp, (const T*)a.kr,             \
        (const T* const*)a.k_chunks, d.chunk_steps, a.vdelta / 2, a.anc, a.plens, a.prompt_len, a.steps, d.beams, \
        d.heads, d.kv_heads, d.group,                                                                  \
        prompt_strides(d), d.max_steps, d.rows)
    switch (d.head_dim) {
        case 64: SEGKV_ROWWISE(64); break;
        case 128: SEGKV_ROWWISE(128); break;
        case 256: SEGKV_ROWWISE(256); break;
        default: return cudaErrorInvalidValue;
    }
#undef SEGKV_ROWWISE
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_sdpa_rowwise(const Dims& d, const SdpaArgs& a, cudaStream_t st) {
    return d.dtype == SEGKV_BF16 ? dispatch<__nv_bfloat16>(d, a, st) : dispatch<__half>(d, a, st);
}

}  // namespace segkv_impl
