/*
 * fp64 CPU oracle for the row-reduction kernel family (RMSNorm forward, last-dim
 * softmax forward, fused cross-entropy forward, LayerNorm forward, row sum).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may call it.  It shares no code,
 * header, table or helper with the CUDA library and is deliberately plain: every
 * function is the textbook definition of the op written as straight loops in
 * double precision, one row at a time, with no blocking, fusion or reordering.
 *
 * What the paper fixes about the ops (it prints no formula for any of them):
 *   - their identity and single-pass/online nature: Table 3 rows "softmax",
 *     "rmsnorm" ("fast rsqrt"), "cross_ent" ("Online log-sum-exp, fused NLL");
 *   - the weight multiply belongs to the RMSNorm epilogue: Section 7.3, Tier 3;
 *   - semantics are those of the PyTorch reference implementation: Section 6
 *     ("Each has a PyTorch reference ... serving as the correctness oracle");
 *   - adversarial inputs to survive: Section 4, Stage 3; bitwise determinism:
 *     Section 4, Stage 4; non-power-of-two sizes: Section 4, Stage 5.
 * Because each op has an exact mathematical definition which a GPU kernel merely
 * evaluates faster, the oracle is that definition:
 *
 *   rmsnorm : ms = (1/D) sum_j x_j^2 ;  y_j = x_j * w_j / sqrt(ms + eps)
 *   softmax : m = max_j x_j ; s = sum_j exp(x_j - m) ; y_j = exp(x_j - m) / s
 *   xent    : t = targets[r]
 *             t == ignore_index      -> loss_r = 0, row not counted
 *             t < 0 or t >= V        -> loss_r = NaN, row counted
 *             otherwise              -> loss_r = (m - x_t) + log(sum_j exp(x_j - m))
 *             loss_mean = (sum over counted rows of loss_r) / n_counted  (0/0 = NaN)
 *   layernorm: mu = mean_j x_j ; var = mean_j (x_j - mu)^2 ;
 *              y_j = (x_j - mu) / sqrt(var + eps) * gamma_j + beta_j   (Table 3 "layernorm")
 *   rowsum  : out_r = sum_j x_rj                                      (Table 3 "reduce")
 *   rope    : pair (2i, 2i+1) at position p rotated by p * base^(-2i/Dh)   (Table 3 "rotary_emb")
 *
 * Inputs are the exact bit patterns the GPU sees (bf16 or fp16 as uint16, or fp32),
 * widened exactly to double; outputs are double and are never rounded.  The *_dt functions
 * take the element type (the paper's harness sweeps FP16 / BF16 / FP32: Section 6); the
 * plain ones are their bf16 case.
 *
 * Readings with no pin in the paper or in mathematics ("parity unpinned", they
 * follow the PyTorch convention): a fully -inf softmax row gives NaN; +inf/NaN
 * inputs propagate per IEEE-754 (a LayerNorm row holding one becomes NaN); eps == 0
 * with an all-zero row gives NaN; an
 * all-ignored batch has mean NaN; an out-of-range target gives NaN for its row.
 * Everything else is pinned by the CPU test-suite (closed forms, invariants,
 * brute force on tiny inputs, an fp64 library cross-check).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE-754 binary32: widening is exact. */
static double bf16_bits_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits.  Widening is exact. */
static double f16_bits_to_double(uint16_t bits)
{
    const int sign = bits >> 15, e = (bits >> 10) & 31, f = bits & 1023;
    double v;
    if (e == 0)       v = ldexp((double)f, -24);                 /* zero and subnormals */
    else if (e == 31) v = f ? NAN : INFINITY;
    else              v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

/* Element types of the *_dt functions (the GPU library's ak_dtype values). */
enum { ORACLE_BF16 = 0, ORACLE_F16 = 1, ORACLE_F32 = 2 };

/* Element i of an array of the given type, widened exactly to double. */
static double load_elem(const void *p, int64_t i, int dtype)
{
    if (dtype == ORACLE_F32) return (double)((const float *)p)[i];
    if (dtype == ORACLE_F16) return f16_bits_to_double(((const uint16_t *)p)[i]);
    return bf16_bits_to_double(((const uint16_t *)p)[i]);
}
static int64_t elem_bytes(int dtype) { return dtype == ORACLE_F32 ? 4 : 2; }

/* Exposed so tests can check the widening itself against known bit patterns. */
void oracle_bf16_to_f64(const uint16_t *src, double *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = bf16_bits_to_double(src[i]);
}
void oracle_f16_to_f64(const uint16_t *src, double *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = f16_bits_to_double(src[i]);
}

/* Threads used by the row loops (rows are independent; each row is sequential, so
 * results do not depend on the thread count).  Returns the count in effect. */
int oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
    return omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}

/* RMSNorm forward (Table 3 "rmsnorm"; Section 7.3 Tier 3 for the fused weight).
 * x: [rows, D] bf16 bits, w: [D] bf16 bits, y: [rows, D] double.
 * eps arrives as the float the GPU entry point receives and is widened. */
void oracle_rmsnorm_dt(const void *x, const void *w, double *y,
                       int64_t rows, int64_t D, float eps, int dtype)
{
    const double eps_d = (double)eps;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const char *xr = (const char *)x + r * D * elem_bytes(dtype);
        double *yr = y + r * D;
        double sumsq = 0.0;
        for (int64_t j = 0; j < D; ++j) {
            double v = load_elem(xr, j, dtype);
            sumsq += v * v;
        }
        double denom = sqrt(sumsq / (double)D + eps_d);
        for (int64_t j = 0; j < D; ++j)
            yr[j] = load_elem(xr, j, dtype) * load_elem(w, j, dtype) / denom;
    }
}
void oracle_rmsnorm(const uint16_t *x, const uint16_t *w, double *y,
                    int64_t rows, int64_t D, float eps)
{
    oracle_rmsnorm_dt(x, w, y, rows, D, eps, ORACLE_BF16);
}

/* LayerNorm forward (Table 3 "layernorm": the paper's kernel is a single-pass Welford; the
 * quantity it evaluates is the textbook one, written here as two plain passes).
 *   mu = (1/D) sum_j x_j ;  var = (1/D) sum_j (x_j - mu)^2   (biased, as in PyTorch)
 *   y_j = (x_j - mu) / sqrt(var + eps) * gamma_j + beta_j
 * x: [rows, D] bf16 bits, gamma/beta: [D] bf16 bits, y: [rows, D] double. */
void oracle_layernorm_dt(const void *x, const void *gamma, const void *beta, double *y,
                         int64_t rows, int64_t D, float eps, int dtype)
{
    const double eps_d = (double)eps;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const char *xr = (const char *)x + r * D * elem_bytes(dtype);
        double *yr = y + r * D;
        double sum = 0.0;
        for (int64_t j = 0; j < D; ++j) sum += load_elem(xr, j, dtype);
        const double mu = sum / (double)D;
        double sq = 0.0;
        for (int64_t j = 0; j < D; ++j) {
            double d = load_elem(xr, j, dtype) - mu;
            sq += d * d;
        }
        const double denom = sqrt(sq / (double)D + eps_d);
        for (int64_t j = 0; j < D; ++j)
            yr[j] = (load_elem(xr, j, dtype) - mu) / denom * load_elem(gamma, j, dtype)
                    + load_elem(beta, j, dtype);
    }
}
void oracle_layernorm(const uint16_t *x, const uint16_t *gamma, const uint16_t *beta, double *y,
                      int64_t rows, int64_t D, float eps)
{
    oracle_layernorm_dt(x, gamma, beta, y, rows, D, eps, ORACLE_BF16);
}

/* Row sum (Table 3 "reduce": hierarchical reduction of each row to one number).
 * x: [rows, D] bf16 bits, out: [rows] double, plain left-to-right sum in double. */
void oracle_rowsum_dt(const void *x, double *out, int64_t rows, int64_t D, int dtype)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const char *xr = (const char *)x + r * D * elem_bytes(dtype);
        double sum = 0.0;
        for (int64_t j = 0; j < D; ++j) sum += load_elem(xr, j, dtype);
        out[r] = sum;
    }
}
void oracle_rowsum(const uint16_t *x, double *out, int64_t rows, int64_t D)
{
    oracle_rowsum_dt(x, out, rows, D, ORACLE_BF16);
}

/* Rotary position embedding forward (Table 3 "rotary_emb": interleaved rotation; Table 4
 * rows "rotary", shape batch x heads x sequence x head_dim).  x: [n_seq, S, Dh] elements of
 * `dtype` (n_seq = batch * heads); the head vector at sequence index s has position
 * p = pos_offset + s, and its pair i = elements (2i, 2i + 1) is rotated by the angle
 *   theta = p * base^(-2i / Dh):
 *   y[2i]     = x[2i] cos(theta) - x[2i + 1] sin(theta)
 *   y[2i + 1] = x[2i] sin(theta) + x[2i + 1] cos(theta)
 * `base` arrives as the float the GPU entry point receives and is widened.  Dh must be even. */
void oracle_rope(const void *x, double *y, int64_t n_seq, int64_t S, int64_t Dh,
                 float base, int64_t pos_offset, int dtype)
{
    const double base_d = (double)base;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_seq * S; ++r) {
        const int64_t s = r % S;
        const double p = (double)(pos_offset + s);
        const char *xr = (const char *)x + r * Dh * elem_bytes(dtype);
        double *yr = y + r * Dh;
        for (int64_t i = 0; i < Dh / 2; ++i) {
            const double theta = p * pow(base_d, -2.0 * (double)i / (double)Dh);
            const double c = cos(theta), sn = sin(theta);
            const double a = load_elem(xr, 2 * i, dtype), b = load_elem(xr, 2 * i + 1, dtype);
            yr[2 * i] = a * c - b * sn;
            yr[2 * i + 1] = a * sn + b * c;
        }
    }
}

/* Last-dim softmax forward (Table 3 "softmax").  A causal mask is part of the data
 * (-inf entries); exp(-inf - m) is exactly 0 for finite m. */
void oracle_softmax_dt(const void *x, double *y, int64_t rows, int64_t D, int dtype)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const char *xr = (const char *)x + r * D * elem_bytes(dtype);
        double *yr = y + r * D;
        double m = -INFINITY;
        int saw_nan = 0;
        for (int64_t j = 0; j < D; ++j) {
            double v = load_elem(xr, j, dtype);
            if (isnan(v)) saw_nan = 1;
            if (v > m) m = v;
        }
        if (saw_nan) m = NAN;
        double s = 0.0;
        for (int64_t j = 0; j < D; ++j)
            s += exp(load_elem(xr, j, dtype) - m);
        for (int64_t j = 0; j < D; ++j)
            yr[j] = exp(load_elem(xr, j, dtype) - m) / s;
    }
}
void oracle_softmax(const uint16_t *x, double *y, int64_t rows, int64_t D)
{
    oracle_softmax_dt(x, y, rows, D, ORACLE_BF16);
}

/* Fused cross-entropy forward (Table 3 "cross_ent": log-sum-exp fused with the
 * negative log-likelihood gather).  loss_rows: [rows] double.  *loss_mean and
 * *n_counted may be NULL.  The loss is formed as (m - x_t) + log(s): both terms are
 * >= 0 (the maximum contributes exp(0) = 1 to s), so loss >= 0 holds structurally. */
void oracle_xent_dt(const void *logits, const int64_t *targets, int64_t ignore_index,
                    double *loss_rows, double *loss_mean, int64_t *n_counted,
                    int64_t rows, int64_t V, int dtype)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const int64_t t = targets[r];
        if (t == ignore_index) { loss_rows[r] = 0.0; continue; }
        if (t < 0 || t >= V)   { loss_rows[r] = NAN; continue; }
        const char *xr = (const char *)logits + r * V * elem_bytes(dtype);
        double m = -INFINITY;
        int saw_nan = 0;
        for (int64_t j = 0; j < V; ++j) {
            double v = load_elem(xr, j, dtype);
            if (isnan(v)) saw_nan = 1;
            if (v > m) m = v;
        }
        if (saw_nan) m = NAN;
        double s = 0.0;
        for (int64_t j = 0; j < V; ++j)
            s += exp(load_elem(xr, j, dtype) - m);
        loss_rows[r] = (m - load_elem(xr, t, dtype)) + log(s);
    }
    /* Mean over counted rows, sequential, in row order. */
    double total = 0.0;
    int64_t count = 0;
    for (int64_t r = 0; r < rows; ++r) {
        if (targets[r] == ignore_index) continue;
        total += loss_rows[r];
        ++count;
    }
    if (n_counted) *n_counted = count;
    if (loss_mean) *loss_mean = (count > 0) ? total / (double)count : NAN;
}
void oracle_xent(const uint16_t *logits, const int64_t *targets, int64_t ignore_index,
                 double *loss_rows, double *loss_mean, int64_t *n_counted,
                 int64_t rows, int64_t V)
{
    oracle_xent_dt(logits, targets, ignore_index, loss_rows, loss_mean, n_counted, rows, V, ORACLE_BF16);
}
