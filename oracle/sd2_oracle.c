/*
 * CPU oracle for the sparse drafter linears.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain definition of what the CUDA library must compute.
 * It is deliberately slow and obvious: fp64, one loop nest, no blocking, no
 * threads, no vector intrinsics.  It shares no code, header, table or helper
 * with the CUDA library and neither includes the other.  Only the tests, the
 * smoke check and the benchmark's cpu_baseline / reference arm may call it;
 * the product never does.
 *
 * What the paper fixes (and all it fixes):
 *   - A pruned drafter's linear layer keeps a fixed binary mask; pruned
 *     parameters are exactly zero and stay zero (Section "Sparse fine-tuning":
 *     the topology is fixed after one-shot pruning).
 *   - A weight matrix W has shape (C_out, C_in) (Appendix "Non-uniform
 *     layer-wise sparsity distributions", outlier-score definition), i.e. a
 *     linear layer computes Y = X W^T.
 *   - A decoder block is a self-attention module followed by a feed-forward
 *     module (Section "Layer pruning"); all decoder-block linears are pruned,
 *     embedding and LM head stay dense (Section "Results", first paragraph).
 * The sparse kernel and compressed representation (Section "Compressed sparse
 * drafters") must reach exactly the dense masked product, only faster, so the
 * oracle is that product written out.
 *
 * Pins (tests/test_oracle_pins.py): exact rational brute force on tiny
 * matrices with exhaustive masks, an integer-exact case, zero / full / identity
 * masks, one-hot activations, linearity, row and column permutations, a
 * library fp64 matmul for the full mask, and the paper's printed 43.87 % MAC
 * reduction for the layer shapes.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

/* bf16 -> fp64: a bf16 pattern is the upper half of an fp32; widening is exact. */
static double bf16_bits_to_f64(uint16_t h)
{
    uint32_t b = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &b, sizeof f);
    return (double)f;
}

/* Is entry (m,k) kept?  With an explicit mask the mask decides (selection, not
 * multiplication: a masked-out weight never takes part, whatever its bits).
 * Without a mask, the entry is kept iff the weight is not +0 / -0. */
static int kept(const uint16_t* W, const uint8_t* mask, int64_t idx)
{
    if (mask) return mask[idx] != 0;
    return (W[idx] & 0x7FFF) != 0;
}

/*
 * Masked linear layer, Y = X (W .* mask)^T.
 *   W    [M*K] bf16 bit patterns, row-major, M = C_out, K = C_in
 *   mask [M*K] bytes (non-zero = kept) or NULL
 *   X    [N*K] bf16 bit patterns, row-major
 *   Y    [N*M] fp64 out:  Y[n,m] = sum over kept k (ascending) of W[m,k] X[n,k]
 *   S    [N*M] fp64 out:  S[n,m] = sum over kept k of |W[m,k] X[n,k]|
 * Each product of two bf16 values is exact in fp64 (16 significant bits).
 */
void sd2o_masked_linear(const uint16_t* W, const uint8_t* mask, const uint16_t* X,
                        int64_t M, int64_t K, int64_t N, double* Y, double* S)
{
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0, mag = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                if (kept(W, mask, m * K + k)) {
                    double p = bf16_bits_to_f64(W[m * K + k]) * bf16_bits_to_f64(X[n * K + k]);
                    acc += p;
                    mag += fabs(p);
                }
            }
            Y[n * M + m] = acc;
            if (S) S[n * M + m] = mag;
        }
    }
}

/* The dense matrix a lossless compressed format must decode to: kept entries
 * keep their bit pattern (-0, subnormals and NaN payloads included), masked
 * out entries read +0 (0x0000). */
void sd2o_roundtrip_ref(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, uint16_t* out)
{
    for (int64_t i = 0; i < M * K; ++i) out[i] = kept(W, mask, i) ? W[i] : (uint16_t)0;
}

/* Number of kept entries. */
int64_t sd2o_nnz(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K)
{
    int64_t c = 0;
    for (int64_t i = 0; i < M * K; ++i) c += kept(W, mask, i) ? 1 : 0;
    return c;
}

/* Feed-forward glue between gate/up and down: t = silu(g) * u in fp64,
 * silu(g) = g / (1 + exp(-g)).  The paper only says a block has a feed-forward
 * module; SwiGLU is the activation of the Llama-3.2 / Qwen-2.5 drafters it
 * prunes.  g, u are bf16 patterns; out is fp64 (unrounded). */
void sd2o_silu_mul(const uint16_t* g, const uint16_t* u, int64_t n, double* out)
{
    for (int64_t i = 0; i < n; ++i) {
        double a = bf16_bits_to_f64(g[i]);
        out[i] = (a / (1.0 + exp(-a))) * bf16_bits_to_f64(u[i]);
    }
}

/* fp64 -> bf16 with round-to-nearest-even on the exact value (finite inputs
 * within bf16's normal range; used to measure glue results in bf16 ulps). */
uint16_t sd2o_f64_to_bf16_rne(double v)
{
    if (v == 0.0) return signbit(v) ? 0x8000 : 0x0000;
    int e;
    double mant = frexp(fabs(v), &e);             /* |v| = mant * 2^e, mant in [0.5,1) */
    int exp_unb = e - 1;                          /* |v| = (2 mant) * 2^(e-1)           */
    if (exp_unb < -126) exp_unb = -126;           /* subnormal spacing                  */
    double ulp = ldexp(1.0, exp_unb - 7);         /* bf16 has 7 fraction bits           */
    double q = fabs(v) / ulp;                     /* exact: power-of-two scaling        */
    double r = nearbyint(q);                      /* default mode: ties to even         */
    double rv = r * ulp;
    float f = (float)rv;                          /* rv has <= 8 significant bits       */
    uint32_t b;
    memcpy(&b, &f, sizeof b);
    uint16_t h = (uint16_t)(b >> 16);
    return signbit(v) ? (uint16_t)(h | 0x8000) : h;
}
