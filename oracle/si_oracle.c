/*
 * SelectInfer selective-FFN oracle (TEST INFRASTRUCTURE ONLY).
 *
 * A plain, slow, float64 CPU statement of what the selective-computation hot path
 * computes.  It is the yardstick the CUDA library is compared against and shares no
 * code, header, table or helper with it.  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may call it; no product path may.
 *
 * What is computed (paper, Section 3 "LLM Profiler": one FFN neuron is one slice of
 * gate_proj / up_proj and the matching slice of down_proj; Section 5 "Selective
 * Computation": only the selected loaded neurons are computed):
 *
 *     y = sum over i in A of  SiLU(w_gate_i . x) * (w_up_i . x) * W_down[:, i]
 *
 * on the FULL weight matrices in PyTorch [out, in] storage
 *     W_gate, W_up : [d_ff, d_model]     (neuron i = row i)
 *     W_down       : [d_model, d_ff]     (neuron i = column i)
 * with GLOBAL neuron ids, so the oracle never sees the packed neuron store and
 * therefore also checks the loader.  Inputs are the 16-bit patterns the GPU sees,
 * widened exactly to float64; nothing is rounded afterwards.  Neurons are taken in
 * ascending id order and every sum runs over ascending indices (set semantics).
 *
 * Pins (tests/test_oracle_pins.py): library float64 dense SwiGLU for A = all neurons,
 * closed-form one-hot neurons with printed SiLU values, x = 0, additivity over
 * disjoint sets, list-order invariance, exact equality with the masked dense loop.
 * The task-accuracy claims of the paper (EM/BLEU/ROUGE) are out of scope: parity
 * unpinned for those, nothing here computes them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { SO_F64 = 0, SO_F16 = 1, SO_BF16 = 2 };

/* IEEE binary16 bit pattern -> double, exact (handles subnormals, inf, nan). */
static double half_bits_to_double(uint16_t b) {
    int sign = (b >> 15) & 1;
    int e = (b >> 10) & 0x1F;
    int m = b & 0x3FF;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -24);              /* subnormal: m * 2^-24 */
    } else if (e == 31) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(m | 0x400), e - 25); /* (1024+m) * 2^(e-15-10) */
    }
    return sign ? -v : v;
}

/* bfloat16 bit pattern -> double, exact: it is the upper half of a binary32. */
static double bf16_bits_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double elem(const void *p, size_t i, int dtype) {
    if (dtype == SO_F64) return ((const double *)p)[i];
    if (dtype == SO_F16) return half_bits_to_double(((const uint16_t *)p)[i]);
    return bf16_bits_to_double(((const uint16_t *)p)[i]);
}

/* SiLU(g) * u, the value that enters down_proj (Section 3). */
static double neuron_activation(const void *Wg, const void *Wu, const void *x, int dtype,
                                int d_model, int64_t i) {
    double g = 0.0, u = 0.0;
    for (int c = 0; c < d_model; ++c) {
        double xc = elem(x, (size_t)c, dtype);
        g += elem(Wg, (size_t)i * d_model + c, dtype) * xc;
        u += elem(Wu, (size_t)i * d_model + c, dtype) * xc;
    }
    return (g / (1.0 + exp(-g))) * u;
}

static int cmp_i32(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * Selective FFN for one token.  A: k global neuron ids (any order, distinct, in range).
 * h_out (optional, may be NULL): receives h_i for the ids in ascending order.
 * Returns 0, or -1 on a bad id / duplicate.
 * threads > 1 spreads the independent per-neuron dot products, and then the output
 * columns, over OpenMP threads; every individual sum keeps its ascending order, so
 * the result is bit-identical to the single-threaded one.
 */
int so_ffn(const void *Wg, const void *Wu, const void *Wd, int dtype, int d_ff, int d_model,
           const void *x, const int32_t *A, int k, double *y, double *h_out, int threads) {
    for (int j = 0; j < d_model; ++j) y[j] = 0.0;
    if (k == 0) return 0;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
    double *h = (double *)malloc(sizeof(double) * (size_t)k);
    memcpy(ids, A, sizeof(int32_t) * (size_t)k);
    qsort(ids, (size_t)k, sizeof(int32_t), cmp_i32);
    int bad = 0;
    for (int t = 0; t < k; ++t) {
        if (ids[t] < 0 || ids[t] >= d_ff) bad = 1;
        if (t > 0 && ids[t] == ids[t - 1]) bad = 1;
    }
    if (bad) { free(ids); free(h); return -1; }
    if (threads < 1) threads = 1;

#pragma omp parallel for num_threads(threads) schedule(static)
    for (int t = 0; t < k; ++t)
        h[t] = neuron_activation(Wg, Wu, x, dtype, d_model, ids[t]);

#pragma omp parallel for num_threads(threads) schedule(static)
    for (int j = 0; j < d_model; ++j) {
        double acc = 0.0;
        for (int t = 0; t < k; ++t)                       /* ascending neuron id */
            acc += h[t] * elem(Wd, (size_t)j * d_ff + ids[t], dtype);
        y[j] = acc;
    }
    if (h_out) memcpy(h_out, h, sizeof(double) * (size_t)k);
    free(ids); free(h);
    return 0;
}

/*
 * Brute-force counterpart: the dense FFN over ALL d_ff neurons in ascending order
 * with h_i forced to +0 where keep[i] == 0.  Adding +-0 to a running float64 sum that
 * started at +0 never changes it, so this must equal so_ffn on {i : keep[i]} exactly.
 */
int so_ffn_dense_masked(const void *Wg, const void *Wu, const void *Wd, int dtype, int d_ff,
                        int d_model, const void *x, const uint8_t *keep, double *y) {
    double *h = (double *)malloc(sizeof(double) * (size_t)d_ff);
    for (int i = 0; i < d_ff; ++i) {
        double a = neuron_activation(Wg, Wu, x, dtype, d_model, i);
        h[i] = keep[i] ? a : 0.0;
    }
    for (int j = 0; j < d_model; ++j) {
        double acc = 0.0;
        for (int i = 0; i < d_ff; ++i) acc += h[i] * elem(Wd, (size_t)j * d_ff + i, dtype);
        y[j] = acc;
    }
    free(h);
    return 0;
}

/*
 * T tokens, each with its own list (masked-union semantics: token t uses exactly its
 * own list, whatever the other tokens selected).  Lists are CSR: offsets[T+1] into A.
 * X: [T, d_model], Y: [T, d_model] float64.  Tokens are independent; threads split
 * inside each token as in so_ffn.
 */
int so_ffn_tokens(const void *Wg, const void *Wu, const void *Wd, int dtype, int d_ff,
                  int d_model, const void *X, int T, const int32_t *A, const int32_t *offsets,
                  double *Y, int threads) {
    size_t esz = (dtype == SO_F64) ? 8 : 2;
    for (int t = 0; t < T; ++t) {
        const char *xt = (const char *)X + (size_t)t * d_model * esz;
        int rc = so_ffn(Wg, Wu, Wd, dtype, d_ff, d_model, xt, A + offsets[t],
                        offsets[t + 1] - offsets[t], Y + (size_t)t * d_model, NULL, threads);
        if (rc) return rc;
    }
    return 0;
}
