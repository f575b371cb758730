/*
 * qmm_oracle.c -- plain CPU oracle (test infrastructure; see qmm_oracle.h).
 *
 * Everything is written as the definition reads: dequantise each weight
 * exactly, multiply, accumulate in fp64 in ascending k.  No blocking, no
 * vector intrinsics, no reordering.  Loops over independent output rows run
 * under OpenMP; nothing else is parallel.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (no -ffast-math).
 */
#include "qmm_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ fp16 */

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* Exact widening of an IEEE binary16 bit pattern (subnormals, zeros, inf, NaN). */
float orc_h2f(uint16_t h)
{
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1Fu;
    uint32_t m = h & 0x3FFu;
    if (e == 0) {
        if (m == 0) return bits_f32(sign);
        /* subnormal: m * 2^-24; normalise */
        int sh = 0;
        while (!(m & 0x400u)) { m <<= 1; ++sh; }
        m &= 0x3FFu;
        return bits_f32(sign | ((uint32_t)(113 - sh) << 23) | (m << 13));
    }
    if (e == 31) return bits_f32(sign | 0x7F800000u | (m << 13));
    return bits_f32(sign | ((e + 112u) << 23) | (m << 13));
}

/* Round to nearest, ties to even; overflow -> inf; gradual underflow. */
uint16_t orc_f2h(float f)
{
    uint32_t x = f32_bits(f);
    uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
    x &= 0x7FFFFFFFu;
    if (x > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);          /* NaN */
    if (x >= 0x47800000u) return (uint16_t)(sign | 0x7C00u);         /* >= 2^16 */
    if (x >= 0x38800000u) {                                          /* >= 2^-14: normal */
        uint32_t h = (((x >> 23) - 112u) << 10) | ((x & 0x7FFFFFu) >> 13);
        uint32_t rem = x & 0x1FFFu;
        if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) ++h;      /* may carry to inf */
        return (uint16_t)(sign | h);
    }
    {
        uint32_t e = x >> 23;
        uint32_t shift = 126u - e;                                    /* >= 14 here */
        uint32_t m, h, rem, half;
        if (shift > 24u) return sign;                                 /* < 2^-25 */
        m = (x & 0x7FFFFFu) | 0x800000u;
        h = m >> shift;
        rem = m & ((1u << shift) - 1u);
        half = 1u << (shift - 1u);
        if (rem > half || (rem == half && (h & 1u))) ++h;
        return (uint16_t)(sign | h);
    }
}

/* --------------------------------------------------------------- formats */

size_t orc_block_bytes(int fmt)
{
    if (fmt == ORC_Q4) return 18;
    if (fmt == ORC_Q5) return 22;
    if (fmt == ORC_Q6) return 26;
    if (fmt == ORC_Q8) return 34;
    return 0;
}

size_t orc_canonical_bytes(int fmt, int64_t N, int64_t K)
{
    if (N <= 0 || K <= 0 || K % 32) return 0;
    return (size_t)N * (size_t)(K / 32) * orc_block_bytes(fmt);
}

static int block_scale_ok(const uint8_t* blk, float* df)
{
    uint16_t d = (uint16_t)(blk[0] | (blk[1] << 8));
    if (((d >> 10) & 0x1Fu) == 31u) return 0;                         /* inf or NaN */
    *df = orc_h2f(d);
    return 1;
}

/* Decode one block into 32 floats: w_i = h2f(d) * (float)q_i. */
static int decode_block(int fmt, const uint8_t* blk, float* w)
{
    float df;
    int i;
    if (!block_scale_ok(blk, &df)) return 1;
    if (fmt == ORC_Q4) {
        for (i = 0; i < 32; ++i) {
            uint8_t byte = blk[2 + i / 2];
            int u = (i & 1) ? (byte >> 4) : (byte & 0x0F);
            w[i] = df * (float)(u - 8);
        }
    } else if (fmt == ORC_Q5) {
        /* d, then 4 bytes of fifth bits (bit i of the little-endian word: element i), then 16 bytes of low nibbles */
        uint32_t hi = (uint32_t)blk[2] | ((uint32_t)blk[3] << 8) | ((uint32_t)blk[4] << 16) | ((uint32_t)blk[5] << 24);
        for (i = 0; i < 32; ++i) {
            uint8_t byte = blk[6 + i / 2];
            int lo = (i & 1) ? (byte >> 4) : (byte & 0x0F);
            int u = lo | (int)(((hi >> i) & 1u) << 4);
            w[i] = df * (float)(u - 16);
        }
    } else if (fmt == ORC_Q6) {
        /* d, then 8 bytes of high bit pairs (byte i/4, bits 2(i%4) and 2(i%4)+1: element i), then 16 bytes of low nibbles */
        for (i = 0; i < 32; ++i) {
            uint8_t byte = blk[10 + i / 2];
            int lo = (i & 1) ? (byte >> 4) : (byte & 0x0F);
            int hi2 = (blk[2 + i / 4] >> (2 * (i % 4))) & 3;
            int u = lo | (hi2 << 4);
            w[i] = df * (float)(u - 32);
        }
    } else {
        for (i = 0; i < 32; ++i) {
            int q = (int)(int8_t)blk[2 + i];
            w[i] = df * (float)q;
        }
    }
    return 0;
}

int orc_quantize(int fmt, const float* w, int64_t N, int64_t K, uint8_t* blocks)
{
    size_t bb = orc_block_bytes(fmt);
    int64_t nb, nblk, g;
    float qmax, qmin;
    if (!bb || !w || !blocks || N <= 0 || K <= 0 || K % 32) return 1;
    nb = K / 32;
    nblk = N * nb;
    qmax = (fmt == ORC_Q4) ? 7.0f : (fmt == ORC_Q5) ? 15.0f : (fmt == ORC_Q6) ? 31.0f : 127.0f;
    qmin = (fmt == ORC_Q4) ? -8.0f : (fmt == ORC_Q5) ? -16.0f : (fmt == ORC_Q6) ? -32.0f : -127.0f;
#pragma omp parallel for schedule(static)
    for (g = 0; g < nblk; ++g) {
        const float* src = w + g * 32;
        uint8_t* blk = blocks + (size_t)g * bb;
        float amax = 0.0f, df;
        uint16_t d;
        int q[32];
        int i;
        for (i = 0; i < 32; ++i) {
            float a = fabsf(src[i]);
            if (a > amax) amax = a;
        }
        d = orc_f2h(amax / qmax);
        df = orc_h2f(d);
        for (i = 0; i < 32; ++i) {
            if (df == 0.0f) {
                q[i] = 0;
            } else {
                float r = nearbyintf(src[i] / df);                    /* ties to even */
                if (r > qmax) r = qmax;
                if (r < qmin) r = qmin;
                q[i] = (int)r;
            }
        }
        blk[0] = (uint8_t)(d & 0xFF);
        blk[1] = (uint8_t)(d >> 8);
        if (fmt == ORC_Q4) {
            for (i = 0; i < 16; ++i)
                blk[2 + i] = (uint8_t)((q[2 * i] + 8) | ((q[2 * i + 1] + 8) << 4));
        } else if (fmt == ORC_Q5) {
            uint32_t hi = 0;
            for (i = 0; i < 32; ++i) hi |= (uint32_t)(((q[i] + 16) >> 4) & 1) << i;
            for (i = 0; i < 4; ++i) blk[2 + i] = (uint8_t)(hi >> (8 * i));
            for (i = 0; i < 16; ++i)
                blk[6 + i] = (uint8_t)(((q[2 * i] + 16) & 15) | (((q[2 * i + 1] + 16) & 15) << 4));
        } else if (fmt == ORC_Q6) {
            for (i = 0; i < 8; ++i) blk[2 + i] = 0;
            for (i = 0; i < 32; ++i) blk[2 + i / 4] |= (uint8_t)((((q[i] + 32) >> 4) & 3) << (2 * (i % 4)));
            for (i = 0; i < 16; ++i)
                blk[10 + i] = (uint8_t)(((q[2 * i] + 32) & 15) | (((q[2 * i + 1] + 32) & 15) << 4));
        } else {
            for (i = 0; i < 32; ++i) blk[2 + i] = (uint8_t)(int8_t)q[i];
        }
    }
    return 0;
}

int orc_dequant(int fmt, const uint8_t* blocks, int64_t N, int64_t K, float* w)
{
    size_t bb = orc_block_bytes(fmt);
    int64_t nblk, g;
    int bad = 0;
    if (!bb || !w || !blocks || N <= 0 || K <= 0 || K % 32) return 1;
    nblk = N * (K / 32);
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (g = 0; g < nblk; ++g)
        bad |= decode_block(fmt, blocks + (size_t)g * bb, w + g * 32);
    return bad;
}

/* -------------------------------------------------------------- products */

/* One output row against M activation rows given as doubles. */
static void row_times(const float* wrow, int64_t K, const double* X, int64_t ldx, int64_t M,
                      double* Y, double* B, int64_t n, int64_t N)
{
    int64_t m, k;
    for (m = 0; m < M; ++m) {
        const double* x = X + m * ldx;
        double s = 0.0, a = 0.0;
        for (k = 0; k < K; ++k) {
            double t = (double)wrow[k] * x[k];
            s += t;
            a += fabs(t);
        }
        Y[m * N + n] = s;
        if (B) B[m * N + n] = a;
    }
}

int orc_gemm_f64(int fmt, const uint8_t* blocks, int64_t N, int64_t K,
                 const double* X, int64_t ldx, int64_t M, double* Y, double* B)
{
    size_t bb = orc_block_bytes(fmt);
    int64_t nb, n;
    int bad = 0;
    if (!bb || !blocks || !X || !Y || N <= 0 || K <= 0 || K % 32 || M < 0 || ldx < K) return 1;
    nb = K / 32;
#pragma omp parallel reduction(| : bad)
    {
        float* wrow = (float*)malloc((size_t)K * sizeof(float));
        if (!wrow) {
            bad |= 1;
        } else {
#pragma omp for schedule(static)
            for (n = 0; n < N; ++n) {
                int64_t b;
                for (b = 0; b < nb; ++b)
                    bad |= decode_block(fmt, blocks + ((size_t)n * nb + b) * bb, wrow + b * 32);
                row_times(wrow, K, X, ldx, M, Y, B, n, N);
            }
            free(wrow);
        }
    }
    return bad;
}

int orc_gemm(int fmt, const uint8_t* blocks, int64_t N, int64_t K,
             const uint16_t* X, int64_t ldx, int64_t M, double* Y, double* B)
{
    double* Xd;
    int64_t m, k;
    int rc;
    if (!X || M < 0 || K <= 0 || ldx < K) return 1;
    Xd = (double*)malloc((size_t)(M > 0 ? M : 1) * (size_t)K * sizeof(double));
    if (!Xd) return 1;
    for (m = 0; m < M; ++m)
        for (k = 0; k < K; ++k) Xd[m * K + k] = (double)orc_h2f(X[m * ldx + k]);
    rc = orc_gemm_f64(fmt, blocks, N, K, Xd, K, M, Y, B);
    free(Xd);
    return rc;
}

int orc_gemv(int fmt, const uint8_t* blocks, int64_t N, int64_t K,
             const uint16_t* x, double* y, double* B)
{
    return orc_gemm(fmt, blocks, N, K, x, K, 1, y, B);
}

/* ------------------------------------------------------------------- MoE */

int orc_route(const float* logits, int64_t T, int64_t E, int64_t topk, int32_t* idx, double* p)
{
    int64_t t;
    int bad = 0;
    if (!logits || !idx || !p || T < 0 || E <= 0 || topk <= 0 || topk > E) return 1;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (t = 0; t < T; ++t) {
        const float* l = logits + t * E;
        char* taken = (char*)calloc((size_t)E, 1);
        int64_t j, e;
        double lmax, den = 0.0;
        if (!taken) { bad |= 1; continue; }
        for (e = 0; e < E; ++e)
            if (!isfinite(l[e])) bad |= 1;
        /* selection: k passes, each takes the largest remaining logit; a strict
         * '>' while scanning upward leaves equal logits to the lower index.   */
        for (j = 0; j < topk; ++j) {
            int64_t best = -1;
            for (e = 0; e < E; ++e) {
                if (taken[e]) continue;
                if (best < 0 || l[e] > l[best]) best = e;
            }
            taken[best] = 1;
            idx[t * topk + j] = (int32_t)best;
        }
        free(taken);
        lmax = (double)l[idx[t * topk]];
        for (j = 0; j < topk; ++j) den += exp((double)l[idx[t * topk + j]] - lmax);
        for (j = 0; j < topk; ++j) p[t * topk + j] = exp((double)l[idx[t * topk + j]] - lmax) / den;
    }
    return bad;
}

int orc_permute(const int32_t* idx, int64_t T, int64_t topk, int64_t E,
                int32_t* perm, int32_t* offsets)
{
    int64_t e, t, j, r = 0;
    if (!idx || !perm || !offsets || T < 0 || topk <= 0 || E <= 0) return 1;
    for (e = 0; e < E; ++e) {
        offsets[e] = (int32_t)r;
        for (t = 0; t < T; ++t)
            for (j = 0; j < topk; ++j)
                if (idx[t * topk + j] == e) perm[r++] = (int32_t)(t * topk + j);
    }
    offsets[E] = (int32_t)r;
    return r == T * topk ? 0 : 1;
}

double orc_silu(double g) { return g / (1.0 + exp(-g)); }

int orc_moe_tokens(int fmt, const float* logits, const uint16_t* X,
                   const uint8_t* w_gate, const uint8_t* w_up, const uint8_t* w_down,
                   int64_t T, int64_t H, int64_t I, int64_t E, int64_t topk,
                   const int32_t* tok, int64_t ntok, double* out)
{
    size_t gu_bytes = orc_canonical_bytes(fmt, I, H);
    size_t dn_bytes = orc_canonical_bytes(fmt, H, I);
    int64_t s;
    int bad = 0;
    if (!gu_bytes || !dn_bytes || !logits || !X || !w_gate || !w_up || !w_down || !tok || !out)
        return 1;
    for (s = 0; s < ntok; ++s) {
        int64_t t = tok[s], j, c, i, k;
        int32_t* idx;
        double *p, *x, *g, *u, *h, *d;
        if (t < 0 || t >= T) return 1;
        idx = (int32_t*)malloc((size_t)topk * sizeof(int32_t));
        p = (double*)malloc((size_t)topk * sizeof(double));
        x = (double*)malloc((size_t)H * sizeof(double));
        g = (double*)malloc((size_t)I * sizeof(double));
        u = (double*)malloc((size_t)I * sizeof(double));
        h = (double*)malloc((size_t)I * sizeof(double));
        d = (double*)malloc((size_t)H * sizeof(double));
        if (!idx || !p || !x || !g || !u || !h || !d) return 1;
        bad |= orc_route(logits + t * E, 1, E, topk, idx, p);
        for (k = 0; k < H; ++k) x[k] = (double)orc_h2f(X[t * H + k]);
        for (c = 0; c < H; ++c) out[s * H + c] = 0.0;
        for (j = 0; j < topk; ++j) {
            int64_t e = idx[j];
            bad |= orc_gemm_f64(fmt, w_gate + (size_t)e * gu_bytes, I, H, x, H, 1, g, NULL);
            bad |= orc_gemm_f64(fmt, w_up + (size_t)e * gu_bytes, I, H, x, H, 1, u, NULL);
            for (i = 0; i < I; ++i) h[i] = orc_silu(g[i]) * u[i];
            bad |= orc_gemm_f64(fmt, w_down + (size_t)e * dn_bytes, H, I, h, I, 1, d, NULL);
            for (c = 0; c < H; ++c) out[s * H + c] += p[j] * d[c];
        }
        free(idx); free(p); free(x); free(g); free(u); free(h); free(d);
    }
    return bad;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
