/*
 * qmm_oracle.h -- plain CPU oracle for block-quantised matrix products.
 *
 * TEST INFRASTRUCTURE ONLY.  This is the slow, obviously-correct statement of
 * what the GPU library computes: weights stored as 32-element blocks (one fp16
 * scale + 4-bit or 8-bit integer codes) are dequantised exactly and multiplied
 * by fp16 activations with fp64 accumulation.  It shares no code, header,
 * table or constant with the CUDA path and must never be linked into it.
 *
 * What the paper fixes: weights stay quantised in memory and are dequantised
 * inside the product (Sec. 3.3, "Kernel Fusion and Specialisation"); decode is
 * the M=1 product, prefill the same product on [seq_len x dim] activations
 * (Sec. 3.4, "Prefill"); Q4 and Q8 are two of the supported formats (Sec. 4.1).
 * The paper gives no block layout, no quantisation formula and no MoE
 * algorithm; those are conventions of this library, stated beside each
 * function below.
 *
 * Pinned by tests that do not depend on this file's own arithmetic:
 * hand-built blocks with known products, integer-exact special cases checked
 * against integer matrix products, brute-force loops on tiny shapes, an
 * independent decoder, exhaustive fp16 round trips and comparison with a
 * library fp16 type.  No function here is "parity unpinned".
 */
#ifndef QMM_ORACLE_H
#define QMM_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_Q4 = 4, ORC_Q5 = 5, ORC_Q6 = 6, ORC_Q8 = 8 };

/* ---- fp16 <-> fp32, bit level (IEEE binary16, round to nearest even) ---- */
float    orc_h2f(uint16_t h);
uint16_t orc_f2h(float f);

/* ---- canonical block format -------------------------------------------- *
 * Q4 block, 18 bytes: uint16 d (fp16 bits, little endian); uint8 qs[16];
 *   element i in [0,32) has code q_i in [-8,7] stored as u_i = q_i + 8;
 *   qs[j] = u_{2j} | (u_{2j+1} << 4).
 * Q8 block, 34 bytes: uint16 d; int8 qs[32] (two's complement).
 * Q5 block, 22 bytes: uint16 d; uint8 qh[4]; uint8 qs[16]; code q_i in [-16,15]
 *   stored as u_i = q_i + 16: qs as in Q4 with the low four bits of u, bit i of
 *   the little-endian 32-bit word qh = the fifth bit of u_i.
 * Q6 block, 26 bytes: uint16 d; uint8 qh[8]; uint8 ql[16]; code q_i in [-32,31]
 *   stored as u_i = q_i + 32: ql as in Q4 with the low four bits of u, bits
 *   2(i%4), 2(i%4)+1 of qh[i/4] = the two high bits of u_i.
 *   (The paper's library spans 2-bit to 16-bit formats, Sec. 3.3 / Sec. 4.1,
 *   and gives no layout for any of them; these two are this library's.)
 * Matrix W[N,K]: row n holds K/32 consecutive blocks, rows consecutive.
 * Dequantised weight: w = h2f(d) * (float)q, which is exact in fp32.       */
size_t orc_block_bytes(int fmt);                    /* 18, 22, 26 or 34; 0 if fmt unknown */
size_t orc_canonical_bytes(int fmt, int64_t N, int64_t K);

/* Quantiser (inputs only; the GPU never quantises).  Per block, in fp32:
 * amax = max|w_i|; d = f2h(amax/QMAX), QMAX = 7 (Q4), 15 (Q5), 31 (Q6) or 127 (Q8);
 * df = h2f(d); df == 0 -> all codes 0; else q_i = clamp(rne(w_i/df)).
 * Returns 0 on success, nonzero on bad arguments.                          */
int orc_quantize(int fmt, const float* w, int64_t N, int64_t K, uint8_t* blocks);

/* blocks -> fp32 W[N,K] row-major.  Returns 0, or nonzero if a scale is
 * inf/NaN or arguments are bad.                                            */
int orc_dequant(int fmt, const uint8_t* blocks, int64_t N, int64_t K, float* w);

/* ---- products ----------------------------------------------------------- *
 * Y[m,n] = sum_k w[n,k] * h2f(X[m*ldx + k])   (fp64, k ascending)
 * B[m,n] = sum_k |w[n,k] * h2f(X[m*ldx + k])| (fp64) -- the tolerance scale.
 * Y and B are [M,N] row-major doubles; B may be NULL.                      */
int orc_gemm(int fmt, const uint8_t* blocks, int64_t N, int64_t K,
             const uint16_t* X, int64_t ldx, int64_t M, double* Y, double* B);
/* The M = 1 case.                                                          */
int orc_gemv(int fmt, const uint8_t* blocks, int64_t N, int64_t K,
             const uint16_t* x, double* y, double* B);
/* Same product with fp64 activations (for MoE stages that must not round). */
int orc_gemm_f64(int fmt, const uint8_t* blocks, int64_t N, int64_t K,
                 const double* X, int64_t ldx, int64_t M, double* Y, double* B);

/* ---- mixture-of-experts pieces ------------------------------------------ *
 * Routing: per token the topk largest logits, larger first, equal logits ->
 * lower expert index first (slot 0 is the arg-max); weights are the softmax
 * over the selected logits only, in fp64.                                  */
int orc_route(const float* logits, int64_t T, int64_t E, int64_t topk,
              int32_t* idx, double* p);
/* Permutation: the T*topk pairs (t,j) sorted by (idx[t,j], t) ascending.
 * perm[r] = t*topk + j of sorted position r; offsets[e] = number of pairs
 * with expert < e; offsets[E] = T*topk.                                    */
int orc_permute(const int32_t* idx, int64_t T, int64_t topk, int64_t E,
                int32_t* perm, int32_t* offsets);
/* silu(g) = g / (1 + exp(-g)), fp64.                                       */
double orc_silu(double g);
/* Whole layer in fp64 with no intermediate rounding:
 * out[t,:] = sum_j p[t,j] * Wdown_e( silu(Wgate_e x_t) * (Wup_e x_t) ),
 * e = idx[t,j].  w_gate/w_up: E matrices [I,H]; w_down: E matrices [H,I];
 * each expert's canonical blocks follow the previous one's.
 * Only tokens listed in tok[0..ntok) are computed; out is [ntok,H].        */
int orc_moe_tokens(int fmt, const float* logits, const uint16_t* X,
                   const uint8_t* w_gate, const uint8_t* w_up, const uint8_t* w_down,
                   int64_t T, int64_t H, int64_t I, int64_t E, int64_t topk,
                   const int32_t* tok, int64_t ntok, double* out);

/* Number of threads the parallel loops use (OpenMP).                       */
int orc_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
