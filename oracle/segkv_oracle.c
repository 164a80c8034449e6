/*
 * CPU float64 oracle for decode attention over a segment KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
 * the GPU library must compute.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may build or call it; the product never does,
 * and it shares no code, header or table with the CUDA sources.
 *
 * What it computes (paper Section 3.3, "Customized SDPA Kernel"): for every
 * beam slot g = b*BW + j and query head h the attention context
 *
 *     out[g,h,:] = softmax( q[g,h,:] . Kt^T / sqrt(D) + bias ) . Vt
 *
 * where Kt / Vt are the prompt rows of request b (stored once per request,
 * Section 3.2) followed by one response row per time step s = 0..t, the row
 * being chosen through the beam-index table ("index select", Section 3.3).
 * The index table is obtained by walking the beam-search parent pointers from
 * the current step back to step 0, which is what re-ordering the whole past
 * cache by Indice_t at every step (Section 3.1, the standard flow of Fig. 1)
 * amounts to.  Prompt part and response part go through ONE softmax: the
 * paper accumulates the two partial contexts into one result (Section 3.3).
 *
 * The oracle deliberately does what the GPU path avoids: it concatenates the
 * selected rows into a private K/V copy per beam and runs textbook attention
 * on it, in double precision, with no blocking, no online softmax, no sharing.
 *
 * Layouts (all contiguous, 16-bit storage passed as raw bit patterns):
 *   q        [BS*BW, H, D]
 *   kp, vp   [BS, P, Hkv, D]          prompt, token-major (Section 3.2)
 *   kr, vr   [T, BS*BW, Hkv, D]       response, sequence-first (Section 3.1)
 *   parent   [T, BS*BW] int32         LOCAL beam id in [0,BW) that slot g
 *                                     extends at step s; row 0 is ignored
 *   slopes   [H] float or NULL        ALiBi slopes (not in the paper; the
 *                                     Bloom workload adds bias slope*(kpos-qpos))
 *
 * Parity pins live in tests/test_oracle_pins.py.  The paper prints no
 * attention output values, so the numerical value of the context is pinned
 * only by closed forms, special cases and brute force, not by a paper number.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F16 = 0, ORACLE_BF16 = 1 };

/* IEEE binary16 -> double, exact. */
static double f16_to_f64(uint16_t h) {
    int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);               /* zero / subnormal */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);          /* (1 + m/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* bfloat16 is the upper half of a binary32. */
static double bf16_to_f64(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double widen(int dtype, uint16_t bits) {
    return dtype == ORACLE_BF16 ? bf16_to_f64(bits) : f16_to_f64(bits);
}

/* Test hook: widen n stored values to double. */
void segkv_oracle_widen(int dtype, const uint16_t* bits, long n, double* out) {
    for (long i = 0; i < n; ++i) out[i] = widen(dtype, bits[i]);
}

/*
 * Beam-index table at step t (Section 3.3, "Index select fusion"): rows[g][s]
 * is the row of the step-s response slab that holds beam slot g's key/value.
 * Walk: slot g itself at step t; the slot it extended at step t-1 is
 * parent[t][g]; and so on down to step 0.  rows is [BS*BW][t+1].
 */
void segkv_oracle_ancestry(const int32_t* parent, int BS, int BW, int t, int32_t* rows) {
    int G = BS * BW;
    for (int g = 0; g < G; ++g) {
        int b = g / BW;
        int cur = g % BW;
        for (int s = t; s >= 0; --s) {
            rows[(long)g * (t + 1) + s] = b * BW + cur;
            if (s > 0) cur = parent[(long)s * G + b * BW + cur];
        }
    }
}

/*
 * Attention context for a list of (g, h) pairs at step t (t = -1: no response
 * rows yet, prompt only).  out is [npairs][D]; probs, if not NULL, receives
 * the softmax row [npairs][P+t+1].  Returns 0, or -1 on a bad argument.
 */
int segkv_oracle_decode(int dtype, int BS, int BW, int H, int Hkv, int D, int P, int t,
                        const uint16_t* q, const uint16_t* kp, const uint16_t* vp,
                        const uint16_t* kr, const uint16_t* vr, const int32_t* parent,
                        const float* slopes, const int32_t* pairs, int npairs,
                        double* out, double* probs) {
    if (BS <= 0 || BW <= 0 || H <= 0 || Hkv <= 0 || H % Hkv || D <= 0 || P < 0 || t < -1) return -1;
    int G = BS * BW;
    int L = P + t + 1;                       /* keys this query attends to */
    if (L <= 0) return -1;
    int group = H / Hkv;                     /* query heads per kv head */
    int fail = 0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int ip = 0; ip < npairs; ++ip) {
        int g = pairs[2 * ip], h = pairs[2 * ip + 1];
        if (g < 0 || g >= G || h < 0 || h >= H) { fail = 1; continue; }
        int b = g / BW, kvh = h / group;
        double* Kt = (double*)malloc(sizeof(double) * (size_t)L * D);
        double* Vt = (double*)malloc(sizeof(double) * (size_t)L * D);
        double* sc = (double*)malloc(sizeof(double) * (size_t)L);
        double* qv = (double*)malloc(sizeof(double) * (size_t)D);

        /* 1. prompt rows of request b: one copy, whatever the beam */
        for (int i = 0; i < P; ++i) {
            long src = (((long)b * P + i) * Hkv + kvh) * D;
            for (int d = 0; d < D; ++d) {
                Kt[(long)i * D + d] = widen(dtype, kp[src + d]);
                Vt[(long)i * D + d] = widen(dtype, vp[src + d]);
            }
        }
        /* 2. response rows: walk the parents from step t down to step 0 */
        int cur = g % BW;
        for (int s = t; s >= 0; --s) {
            int row = b * BW + cur;
            long src = (((long)s * G + row) * Hkv + kvh) * D;
            for (int d = 0; d < D; ++d) {
                Kt[(long)(P + s) * D + d] = widen(dtype, kr[src + d]);
                Vt[(long)(P + s) * D + d] = widen(dtype, vr[src + d]);
            }
            if (s > 0) cur = parent[(long)s * G + row];
        }
        /* 3. scores = q.K / sqrt(D) + bias */
        for (int d = 0; d < D; ++d) qv[d] = widen(dtype, q[((long)g * H + h) * D + d]);
        double inv = 1.0 / sqrt((double)D);
        int qpos = L - 1;                    /* position of the newest token */
        double mx = -INFINITY;
        for (int i = 0; i < L; ++i) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qv[d] * Kt[(long)i * D + d];
            double s = dot * inv;
            if (slopes) s += (double)slopes[h] * (double)(i - qpos);
            sc[i] = s;
            if (s > mx) mx = s;
        }
        /* 4. softmax, then the weighted sum of value rows */
        double den = 0.0;
        for (int i = 0; i < L; ++i) { sc[i] = exp(sc[i] - mx); den += sc[i]; }
        for (int i = 0; i < L; ++i) sc[i] /= den;
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int i = 0; i < L; ++i) acc += sc[i] * Vt[(long)i * D + d];
            out[(long)ip * D + d] = acc;
        }
        if (probs) memcpy(probs + (long)ip * L, sc, sizeof(double) * (size_t)L);
        free(Kt); free(Vt); free(sc); free(qv);
    }
    return fail ? -1 : 0;
}

/*
 * Prefill attention (Section 3.1 / 3.3: the prefill kernel is the special case of the decode
 * kernel that sees only query and prompt key/value, batch-first in and out): causal
 * self-attention of every prompt position over the positions up to itself,
 *     out[b,i,h,:] = softmax_{j<=i}( q[b,i,h,:] . k[b,j,kvh,:] / sqrt(D) + bias ) . v[b,j,kvh,:]
 * with bias = slope[h] * (j - i) when slopes are given.  q, out: [BS, N, H, D]; k, v: [BS, N, Hkv, D]
 * (token-major, 16-bit storage as raw bits).  `rows` lists (b, i, h) triples; out is [nrows][D].
 */
int segkv_oracle_prefill(int dtype, int BS, int N, int H, int Hkv, int D, const uint16_t* q,
                         const uint16_t* k, const uint16_t* v, const float* slopes, const int32_t* rows,
                         int nrows, double* out) {
    if (BS <= 0 || N <= 0 || H <= 0 || Hkv <= 0 || H % Hkv || D <= 0) return -1;
    int group = H / Hkv, fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int ir = 0; ir < nrows; ++ir) {
        int b = rows[3 * ir], i = rows[3 * ir + 1], h = rows[3 * ir + 2];
        if (b < 0 || b >= BS || i < 0 || i >= N || h < 0 || h >= H) { fail = 1; continue; }
        int kvh = h / group, L = i + 1;
        double* sc = (double*)malloc(sizeof(double) * (size_t)L);
        double inv = 1.0 / sqrt((double)D), mx = -INFINITY;
        for (int j = 0; j < L; ++j) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += widen(dtype, q[(((long)b * N + i) * H + h) * D + d]) *
                       widen(dtype, k[(((long)b * N + j) * Hkv + kvh) * D + d]);
            double s = dot * inv;
            if (slopes) s += (double)slopes[h] * (double)(j - i);
            sc[j] = s;
            if (s > mx) mx = s;
        }
        double den = 0.0;
        for (int j = 0; j < L; ++j) { sc[j] = exp(sc[j] - mx); den += sc[j]; }
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int j = 0; j < L; ++j) acc += sc[j] / den * widen(dtype, v[(((long)b * N + j) * Hkv + kvh) * D + d]);
            out[(long)ir * D + d] = acc;
        }
        free(sc);
    }
    return fail ? -1 : 0;
}

/*
 * KV-cache sizes in bytes (Section 3.2).  Eq. 1: one token's K and V over all
 * layers.  Eq. 2: the standard contiguous cache, prompt copied per beam.
 * Eq. 3: the segment cache, prompt once per request, response capacity grown
 * in chunks of `chunk` steps (16 in the paper).
 */
double segkv_oracle_cache_token(int L, int H, int D, int elem_bytes) {
    return 2.0 * L * H * D * elem_bytes;
}
double segkv_oracle_cache_standard(int BS, int BW, long n_prompt, long n_response, double token) {
    return (double)BS * BW * (double)(n_prompt + n_response) * token;
}
double segkv_oracle_cache_segment(int BS, int BW, long n_prompt, long n_response, int chunk, double token) {
    long cap = ((n_response + chunk - 1) / chunk) * chunk;
    return (double)BS * ((double)n_prompt + (double)BW * (double)cap) * token;
}

int segkv_oracle_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
