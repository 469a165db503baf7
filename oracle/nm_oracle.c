/*
 * nm_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the NeuralMatrix forward pass: every
 * nonlinear operator is a piecewise-linear (PWL) table evaluated as
 * y = k[s]*x + b[s], every linear operator is a textbook loop nest.  Written
 * from the paper alone; it shares no source, header, table or helper with
 * the CUDA library and must only be called from tests, the smoke check and
 * the CPU-baseline leg of the benchmark.
 *
 * What each routine follows:
 *   nmo_table_secant    Section 3.2.1 "Post-Training Approximation" (equal
 *                       length, continuous segments) + Algorithm 3 line 1
 *                       (k = secant slope, b = f(x_i) - k*x_i).
 *   nmo_table_bias_correct  Algorithm 3 lines 2-3 (shift b by the mean error).
 *   nmo_hsize_startpoints   Algorithm 2 (merge primary segments).
 *   nmo_pwl_eval*       the "PWL calculation" paragraph of Section 3.2
 *                       (segment matrix S, gather K and B, Y = X.K + B) with
 *                       the out-of-range rule of Section 3.2.1 (inputs outside
 *                       the range reuse the first / last segment's k and b).
 *   nmo_linear          Section 3.1: a linear operator is a matrix product
 *                       plus matrix adds.
 *   nmo_attention, nmo_layernorm, nmo_layernorm_sqrt_recip, nmo_encoder_layer
 *                       the BERT encoder layer of Section 5 with exp, 1/x,
 *                       rsqrt and GELU replaced by PWL tables.
 *   nmo_linear_i8       the INT8 evaluation of Section 5: exact integer
 *                       accumulation, then a strict fp32 epilogue.
 *   nmo_attention_i8    the INT8 evaluation extended to the two matrix products of
 *                       attention (Section 5 evaluates whole INT8 networks): exact
 *                       integer scores and integer P.V, strict fp32 in between.
 *   nmo_fake_quant      the same evaluation at definition level: a tensor is
 *                       replaced by the value its int8 code stands for,
 *                       scale * clamp(rint(x / scale), -127, 127), in fp64.
 *   nmo_antiderivative  the closed-form integrals Algorithm 3's segment mean
 *                       uses (exported so that each can be pinned on its own).
 *   nmo_conv2d_nhwc, nmo_maxpool_nhwc, nmo_avgpool_nhwc
 *                       Section 3.1 (convolution is a linear operator) for
 *                       the ResNet-shaped workload; ReLU is a 2-segment table.
 *
 * Readings where the paper is silent are listed in the design notes of the
 * repository; the ones visible here: GELU is the erf form; the segment index
 * is taken in fp32 with one fused multiply-add (so that a GPU and a CPU take
 * the same integer decision); variance is the biased one; softmax subtracts
 * the final row maximum before the PWL exponential.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC nm_oracle.c -lm
 * (-ffp-contract=off: no implicit fused multiply-adds; the only fused ones
 * are the explicit fmaf() calls of the fp32 index / int8 epilogue contract).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum {
    NMO_F_GELU = 0, NMO_F_EXP = 1, NMO_F_RECIP = 2, NMO_F_RSQRT = 3,
    NMO_F_RELU = 4, NMO_F_SQRT = 5, NMO_F_IDENTITY = 6
};

/* A PWL operator as the oracle sees it: n equal segments on [x_min, x_max]
 * with fp32 slopes/intercepts, or -- when exact_func >= 0 -- the exact
 * nonlinearity itself (used only to report approximation error). */
typedef struct {
    int32_t n;
    float x_min;
    float x_max;
    const float* k;
    const float* b;
    int32_t exact_func;
} nmo_pwl;

int nmo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- the exact nonlinearities ------------------------------------------------ */

double nmo_exact(int func, double x)
{
    switch (func) {
    case NMO_F_GELU:     return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));
    case NMO_F_EXP:      return exp(x);
    case NMO_F_RECIP:    return 1.0 / x;
    case NMO_F_RSQRT:    return 1.0 / sqrt(x);
    case NMO_F_RELU:     return x > 0.0 ? x : 0.0;
    case NMO_F_SQRT:     return sqrt(x);
    case NMO_F_IDENTITY: return x;
    default:             return NAN;
    }
}

/* antiderivative F with F' = f, for the segment mean of Algorithm 3 */
static double antiderivative(int func, double x);
double nmo_antiderivative(int func, double x) { return antiderivative(func, x); }
static double antiderivative(int func, double x)
{
    switch (func) {
    case NMO_F_GELU: {
        /* integral of x*Phi(x): 0.5*(x^2-1)*Phi(x) + 0.5*x*phi(x) */
        double Phi = 0.5 * (1.0 + erf(x / sqrt(2.0)));
        double phi = exp(-0.5 * x * x) / sqrt(2.0 * M_PI);
        return 0.5 * (x * x - 1.0) * Phi + 0.5 * x * phi;
    }
    case NMO_F_EXP:      return exp(x);
    case NMO_F_RECIP:    return log(x);
    case NMO_F_RSQRT:    return 2.0 * sqrt(x);
    case NMO_F_RELU:     return x > 0.0 ? 0.5 * x * x : 0.0;
    case NMO_F_SQRT:     return (2.0 / 3.0) * x * sqrt(x);
    case NMO_F_IDENTITY: return 0.5 * x * x;
    default:             return NAN;
    }
}

/* ---- table construction ------------------------------------------------------ */

/* Section 3.2.1 + Algorithm 3 line 1: n segments of equal length h on
 * [x_min, x_max]; on segment i (start x_i = x_min + i*h) the line through
 * (x_i, f(x_i)) and (x_{i+1}, f(x_{i+1})).  fp64 throughout, rounded to fp32
 * once at the end. */
int nmo_table_secant(int func, int n, double x_min, double x_max, float* k, float* b)
{
    if (n < 1 || !(x_max > x_min)) return -1;
    double h = (x_max - x_min) / (double)n;
    for (int i = 0; i < n; ++i) {
        double xi = x_min + (double)i * h;
        double xj = x_min + (double)(i + 1) * h;
        double fi = nmo_exact(func, xi);
        double fj = nmo_exact(func, xj);
        double ki = (fj - fi) / (xj - xi);
        double bi = fi - ki * xi;
        k[i] = (float)ki;
        b[i] = (float)bi;
    }
    return 0;
}

/* Same lines on arbitrary start points xs[0..n] (xs[n] is the end of the last
 * segment); used with the start-point set of Algorithm 2.  fp64 out. */
int nmo_table_secant_points(int func, int n, const double* xs, double* k, double* b)
{
    for (int i = 0; i < n; ++i) {
        double fi = nmo_exact(func, xs[i]);
        double fj = nmo_exact(func, xs[i + 1]);
        k[i] = (fj - fi) / (xs[i + 1] - xs[i]);
        b[i] = fi - k[i] * xs[i];
    }
    return 0;
}

/* Algorithm 3 lines 2-3: dE = mean of f over the segment minus the mean of the
 * secant line (= the average of its two end values); the intercept is moved
 * by dE when |dE| exceeds e_th (the reading the prose of Section 3.2.3 gives;
 * the printed comparison is the other way round). dE is returned per segment. */
int nmo_table_bias_correct(int func, int n, const double* xs, double e_th, double* b, double* dE)
{
    for (int i = 0; i < n; ++i) {
        double x0 = xs[i], x1 = xs[i + 1];
        double mean_f = (antiderivative(func, x1) - antiderivative(func, x0)) / (x1 - x0);
        double d = mean_f - 0.5 * (nmo_exact(func, x0) + nmo_exact(func, x1));
        dE[i] = d;
        if (fabs(d) > e_th) b[i] += d;
    }
    return 0;
}

/* Algorithm 2: walk the range in primary steps dLx; a primary segment whose
 * slope differs from the slope remembered at the last kept start point by more
 * than dK_th opens a new segment there.  Returns the number of start points
 * written to xs (xs[0] = r_min); at most max_pts. */
int nmo_hsize_startpoints(int func, double dLx, double dK_th, double r_min, double r_max,
                          double* xs, int max_pts)
{
    int cnt = 0;
    if (max_pts < 1) return -1;
    xs[cnt++] = r_min;
    double x = r_min + dLx;
    double kref = (nmo_exact(func, x) - nmo_exact(func, r_min)) / dLx;
    /* compare against r_max with a half-step guard so that a range that is a
     * whole number of primary steps is not overrun by rounding */
    while (x < r_max - 0.5 * dLx * 1e-9) {
        double ki = (nmo_exact(func, x + dLx) - nmo_exact(func, x)) / dLx;
        if (fabs(ki - kref) > dK_th) {
            if (cnt >= max_pts) return -1;
            xs[cnt++] = x;
            kref = ki;
        }
        x += dLx;
    }
    return cnt;
}

/* ---- PWL evaluation ---------------------------------------------------------- */

/* The fp32 index contract: inv_h and off are computed in fp64 from the fp32
 * range ends and rounded once; u = fmaf(x, inv_h, off) is one correctly
 * rounded fp32 operation; the segment is floor(u) clamped to [0, n-1]
 * (Section 3.2.1: inputs beyond the range use the end segments' parameters).
 * NaN selects segment 0 (and then propagates through k*x+b). */
static void index_constants(const nmo_pwl* t, float* inv_h, float* off)
{
    double span = (double)t->x_max - (double)t->x_min;
    *inv_h = (float)((double)t->n / span);
    *off = (float)(-(double)t->x_min * (double)t->n / span);
}

int32_t nmo_segment_index(const nmo_pwl* t, float x)
{
    float inv_h, off;
    index_constants(t, &inv_h, &off);
    float u = fmaf(x, inv_h, off);
    if (!(u >= 0.0f)) return 0; /* negative or NaN */
    float fl = floorf(u);
    if (fl >= (float)(t->n - 1)) return t->n - 1;
    return (int32_t)fl;
}

/* y = k[s]*x + b[s] in fp64; the index sees x rounded to fp32. */
static double pwl_one(const nmo_pwl* t, double x, int32_t* idx_out)
{
    if (t->exact_func >= 0) {
        if (idx_out) *idx_out = -1;
        return nmo_exact(t->exact_func, x);
    }
    int32_t s = nmo_segment_index(t, (float)x);
    if (idx_out) *idx_out = s;
    return (double)t->k[s] * x + (double)t->b[s];
}

void nmo_pwl_eval(const nmo_pwl* t, const double* x, int64_t count, double* y, int32_t* idx)
{
    for (int64_t i = 0; i < count; ++i) y[i] = pwl_one(t, x[i], idx ? &idx[i] : NULL);
}

/* strict fp32 evaluation: y = fmaf(k[s], x, b[s]) */
void nmo_pwl_eval_f32(const nmo_pwl* t, const float* x, int64_t count, float* y, int32_t* idx)
{
    for (int64_t i = 0; i < count; ++i) {
        int32_t s = nmo_segment_index(t, x[i]);
        if (idx) idx[i] = s;
        y[i] = fmaf(t->k[s], x[i], t->b[s]);
    }
}

/* ---- linear operator (Section 3.1) ------------------------------------------- */

/* out[m][j] = PWL( sum_c A[m][c]*W[j][c] + bias[j] ) + residual[m][j]
 * A is [M,K] (row stride lda), W is [N,K] (row stride ldw).  Order of the
 * epilogue: bias, then the table, then the residual add. */
void nmo_linear(const double* A, int64_t lda, const double* W, int64_t ldw,
                const double* bias, const double* residual, int64_t ldr,
                int64_t M, int64_t N, int64_t K, const nmo_pwl* t,
                double* out, int64_t ldo, int32_t* idx_out)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int64_t c = 0; c < K; ++c) acc += A[m * lda + c] * W[j * ldw + c];
            if (bias) acc += bias[j];
            int32_t s = -1;
            if (t) acc = pwl_one(t, acc, &s);
            if (idx_out) idx_out[m * N + j] = s;
            if (residual) acc += residual[m * ldr + j];
            out[m * ldo + j] = acc;
        }
    }
}

/* ---- attention --------------------------------------------------------------- */

/* Q, K, V: element (batch bi, token i, head hd, channel c) at
 * base[bi*stride_b + i*stride_t + hd*d + c].  out is [B*L, h*d] row-major.
 * Per query row: s_j = scale * <q_i, k_j>; m = max_j s_j; e_j = PWLexp(s_j - m);
 * sigma = sum_j e_j; r = PWLrecip(sigma); o_i = sum_j (e_j * r) * v_j. */
void nmo_attention(const double* Q, const double* Kp, const double* V,
                   int64_t stride_b, int64_t stride_t,
                   int32_t B, int32_t L, int32_t h, int32_t d, double scale,
                   const nmo_pwl* t_exp, const nmo_pwl* t_recip, double* out)
{
    int64_t rows = (int64_t)B * h * L;
#pragma omp parallel
    {
        double* e = (double*)malloc(sizeof(double) * (size_t)L);
#pragma omp for schedule(static)
        for (int64_t row = 0; row < rows; ++row) {
            int64_t bi = row / ((int64_t)h * L);
            int64_t hd = (row / L) % h;
            int64_t i = row % L;
            const double* q = Q + bi * stride_b + i * stride_t + hd * d;
            double m = -INFINITY;
            for (int64_t j = 0; j < L; ++j) {
                const double* kk = Kp + bi * stride_b + j * stride_t + hd * d;
                double s = 0.0;
                for (int c = 0; c < d; ++c) s += q[c] * kk[c];
                s *= scale;
                e[j] = s;
                if (s > m) m = s;
            }
            double sigma = 0.0;
            for (int64_t j = 0; j < L; ++j) {
                e[j] = pwl_one(t_exp, e[j] - m, NULL);
                sigma += e[j];
            }
            double r = pwl_one(t_recip, sigma, NULL);
            double* o = out + (bi * L + i) * ((int64_t)h * d) + hd * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t j = 0; j < L; ++j) {
                const double* vv = V + bi * stride_b + j * stride_t + hd * d;
                double p = e[j] * r;
                for (int c = 0; c < d; ++c) o[c] += p * vv[c];
            }
        }
        free(e);
    }
}

/* ---- LayerNorm --------------------------------------------------------------- */

/* mu = mean(z); v = mean((z-mu)^2) (biased); r = PWLrsqrt(v + eps);
 * y = (z - mu) * r * gamma + beta */
void nmo_layernorm(const double* z, const double* gamma, const double* beta,
                   int64_t rows, int32_t H, double eps, const nmo_pwl* t_rsqrt, double* y)
{
#pragma omp parallel for schedule(static)
    for (int64_t r0 = 0; r0 < rows; ++r0) {
        const double* zr = z + r0 * H;
        double mu = 0.0;
        for (int c = 0; c < H; ++c) mu += zr[c];
        mu /= (double)H;
        double v = 0.0;
        for (int c = 0; c < H; ++c) v += (zr[c] - mu) * (zr[c] - mu);
        v /= (double)H;
        double r = pwl_one(t_rsqrt, v + eps, NULL);
        for (int c = 0; c < H; ++c) y[r0 * H + c] = (zr[c] - mu) * r * gamma[c] + beta[c];
    }
}

/* The same LayerNorm with the reciprocal square root taken as the paper's own two
 * functions (Section 3.2.2 lists sqrt(x) and 1/x): r = PWLrecip(PWLsqrt(v + eps)). */
void nmo_layernorm_sqrt_recip(const double* z, const double* gamma, const double* beta,
                              int64_t rows, int32_t H, double eps, const nmo_pwl* t_sqrt,
                              const nmo_pwl* t_recip, double* y)
{
#pragma omp parallel for schedule(static)
    for (int64_t r0 = 0; r0 < rows; ++r0) {
        const double* zr = z + r0 * H;
        double mu = 0.0;
        for (int c = 0; c < H; ++c) mu += zr[c];
        mu /= (double)H;
        double v = 0.0;
        for (int c = 0; c < H; ++c) v += (zr[c] - mu) * (zr[c] - mu);
        v /= (double)H;
        double sd = pwl_one(t_sqrt, v + eps, NULL);
        double r = pwl_one(t_recip, sd, NULL);
        for (int c = 0; c < H; ++c) y[r0 * H + c] = (zr[c] - mu) * r * gamma[c] + beta[c];
    }
}

/* ---- one post-LN encoder layer ------------------------------------------------ */

/* x [T,H], T = B*L.  Wqkv [3H,H] (rows 0..H-1 produce Q, H..2H-1 K, 2H..3H-1 V;
 * head hd owns channels hd*d..hd*d+d-1 of each), Wo [H,H], W1 [F,H], W2 [H,F].
 *   qkv = x Wqkv^T + bqkv ;  a = Attention(qkv)
 *   x1  = LN1(x + a Wo^T + bo)
 *   g   = PWLgelu(x1 W1^T + b1)
 *   y   = LN2(x1 + g W2^T + b2) */
int nmo_encoder_layer(const double* x, int32_t B, int32_t L, int32_t H, int32_t h, int32_t F,
                      const double* Wqkv, const double* bqkv, const double* Wo, const double* bo,
                      const double* g1, const double* be1, const double* W1, const double* b1,
                      const double* W2, const double* b2, const double* g2, const double* be2,
                      double eps, const nmo_pwl* t_gelu, const nmo_pwl* t_exp,
                      const nmo_pwl* t_recip, const nmo_pwl* t_rsqrt, double* y)
{
    int64_t T = (int64_t)B * L;
    int32_t d = H / h;
    double* qkv = (double*)malloc(sizeof(double) * (size_t)(T * 3 * H));
    double* a = (double*)malloc(sizeof(double) * (size_t)(T * H));
    double* z = (double*)malloc(sizeof(double) * (size_t)(T * H));
    double* x1 = (double*)malloc(sizeof(double) * (size_t)(T * H));
    double* g = (double*)malloc(sizeof(double) * (size_t)(T * F));
    if (!qkv || !a || !z || !x1 || !g) { free(qkv); free(a); free(z); free(x1); free(g); return -1; }

    nmo_linear(x, H, Wqkv, H, bqkv, NULL, 0, T, 3 * H, H, NULL, qkv, 3 * H, NULL);
    nmo_attention(qkv, qkv + H, qkv + 2 * H, (int64_t)L * 3 * H, 3 * H, B, L, h, d,
                  1.0 / sqrt((double)d), t_exp, t_recip, a);
    nmo_linear(a, H, Wo, H, bo, x, H, T, H, H, NULL, z, H, NULL);
    nmo_layernorm(z, g1, be1, T, H, eps, t_rsqrt, x1);
    nmo_linear(x1, H, W1, H, b1, NULL, 0, T, F, H, t_gelu, g, F, NULL);
    nmo_linear(g, F, W2, F, b2, x1, H, T, H, F, NULL, z, H, NULL);
    nmo_layernorm(z, g2, be2, T, H, eps, t_rsqrt, y);

    free(qkv); free(a); free(z); free(x1); free(g);
    return 0;
}

/* ---- INT8 linear: exact integers, then a strict fp32 epilogue ------------------ */

/* acc[m][j] = sum_c Aq[m][c]*Wq[j][c]                      (int32, exact)
 * x   = fmaf((float)acc, a_scale*w_scale[j], bias[j])      (one fp32 multiply, one fma)
 * s   = segment index of x (fp32 contract above);  y = fmaf(k[s], x, b[s])
 * y  += residual[m][j]  (fp32 add) when a residual is given
 * q   = clamp(rintf(y * inv_out_scale), -127, 127)         (ties to even)
 * Any of acc/idx/y/q may be NULL. t may be NULL (no table: y = x). */
void nmo_linear_i8(const int8_t* Aq, const int8_t* Wq, int64_t M, int64_t N, int64_t K,
                   float a_scale, const float* w_scale, const float* bias,
                   const float* residual, const nmo_pwl* t, float inv_out_scale,
                   int32_t* acc_out, int32_t* idx_out, float* y_out, int8_t* q_out)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t j = 0; j < N; ++j) {
            int32_t acc = 0;
            for (int64_t c = 0; c < K; ++c) acc += (int32_t)Aq[m * K + c] * (int32_t)Wq[j * K + c];
            float sc = a_scale * w_scale[j];
            float x = fmaf((float)acc, sc, bias ? bias[j] : 0.0f);
            int32_t s = -1;
            float yv = x;
            if (t) {
                s = nmo_segment_index(t, x);
                yv = fmaf(t->k[s], x, t->b[s]);
            }
            if (residual) yv = yv + residual[m * N + j];
            if (acc_out) acc_out[m * N + j] = acc;
            if (idx_out) idx_out[m * N + j] = s;
            if (y_out) y_out[m * N + j] = yv;
            if (q_out) {
                float r = rintf(yv * inv_out_scale);
                if (r > 127.0f) r = 127.0f;
                if (r < -127.0f) r = -127.0f;
                q_out[m * N + j] = (int8_t)r;
            }
        }
    }
}

/* ---- INT8 attention: both matrix products on integers -------------------------- */

/* Q, K, V are int8 codes with per-tensor scales s_q, s_k, s_v; element (batch bi, token i, head hd,
 * channel c) at base[bi*stride_b + i*stride_t + hd*d + c].  Per (batch, head, query row i), strict fp32
 * between the integer parts (every step one correctly rounded fp32 operation, so that a GPU can take the
 * same integer decisions):
 *   acc_j  = sum_c Q[i,c]*K[j,c]                          int32, exact
 *   sc     = (s_q * s_k) * scale                          two fp32 multiplies
 *   m      = max_j acc_j;  neg = -((float)m * sc)         the row maximum, taken on the integers (sc > 0)
 *   x_j    = fmaf((float)acc_j, sc, neg)                  scaled score minus the row maximum, one rounding
 *   e_j    = fmaf(k[s], x_j, b[s]), s = segment of x_j    PWL exponential, fp32 contract
 *   p_j    = clamp(rintf(e_j * 127), -127, 127)           the probability as an int8 code of scale 1/127
 *   sigma  = (float)(sum_j p_j) * (1/127)                 the row sum OF THE CODES (an integer sum: exact)
 *   r      = fmaf(kr[t], sigma, br[t]), t = segment       PWL reciprocal
 *   o_c    = sum_j p_j*V[j,c]                             int32, exact
 *   out_c  = ((float)o_c * (s_v * (1/127))) * r           fp32
 * The paper gives no INT8 scheme; this is the reading taken (probabilities quantised with the fixed scale
 * 1/127 because they lie in [0, 1], rows normalised by the sum of what is actually multiplied into V).
 * out is fp32 [B*L, h*d].  acc_dump / p_dump / oacc_dump (any may be NULL): scores [B,h,L,L] int32, codes
 * [B,h,L,L] int8, integer P.V [B*L, h*d] int32. */
void nmo_attention_i8(const int8_t* Q, const int8_t* Kp, const int8_t* V, int64_t stride_b, int64_t stride_t,
                      int32_t B, int32_t L, int32_t h, int32_t d, float s_q, float s_k, float s_v, float scale,
                      const nmo_pwl* t_exp, const nmo_pwl* t_recip, float* out, int32_t* acc_dump,
                      int8_t* p_dump, int32_t* oacc_dump)
{
    const float sc = (s_q * s_k) * scale;
    const float inv127 = 1.0f / 127.0f;
    const float c1 = s_v * inv127;
    int64_t rows = (int64_t)B * h * L;
#pragma omp parallel
    {
        int32_t* acc = (int32_t*)malloc(sizeof(int32_t) * (size_t)L);
        int8_t* p = (int8_t*)malloc((size_t)L);
#pragma omp for schedule(static)
        for (int64_t row = 0; row < rows; ++row) {
            int64_t bi = row / ((int64_t)h * L);
            int64_t hd = (row / L) % h;
            int64_t i = row % L;
            const int8_t* q = Q + bi * stride_b + i * stride_t + hd * d;
            int32_t m = INT32_MIN;
            for (int64_t j = 0; j < L; ++j) {
                const int8_t* kk = Kp + bi * stride_b + j * stride_t + hd * d;
                int32_t a = 0;
                for (int c = 0; c < d; ++c) a += (int32_t)q[c] * (int32_t)kk[c];
                acc[j] = a;
                if (a > m) m = a;
            }
            float neg = -((float)m * sc);
            int32_t isum = 0;
            for (int64_t j = 0; j < L; ++j) {
                float x = fmaf((float)acc[j], sc, neg);
                int32_t s = nmo_segment_index(t_exp, x);
                float e = fmaf(t_exp->k[s], x, t_exp->b[s]);
                float rr = rintf(e * 127.0f);
                if (rr > 127.0f) rr = 127.0f;
                if (!(rr >= -127.0f)) rr = -127.0f;   /* also NaN, as in the quantiser above */
                p[j] = (int8_t)rr;
                isum += p[j];
            }
            float sigma = (float)isum * inv127;
            int32_t t = nmo_segment_index(t_recip, sigma);
            float r = fmaf(t_recip->k[t], sigma, t_recip->b[t]);
            float* o = out + (bi * L + i) * ((int64_t)h * d) + hd * d;
            for (int c = 0; c < d; ++c) {
                int32_t oa = 0;
                for (int64_t j = 0; j < L; ++j)
                    oa += (int32_t)p[j] * (int32_t)V[bi * stride_b + j * stride_t + hd * d + c];
                if (oacc_dump) oacc_dump[(bi * L + i) * ((int64_t)h * d) + hd * d + c] = oa;
                o[c] = ((float)oa * c1) * r;
            }
            if (acc_dump) memcpy(acc_dump + row * L, acc, sizeof(int32_t) * (size_t)L);
            if (p_dump) memcpy(p_dump + row * L, p, (size_t)L);
        }
        free(acc);
        free(p);
    }
}

/* symmetric quantisation of a tensor with a given scale: q = clamp(rintf(x*inv_scale)) */
void nmo_quantize_i8(const float* x, int64_t count, float inv_scale, int8_t* q)
{
    for (int64_t i = 0; i < count; ++i) {
        float r = rintf(x[i] * inv_scale);
        if (r > 127.0f) r = 127.0f;
        if (r < -127.0f) r = -127.0f;
        q[i] = (int8_t)r;
    }
}

/* Definition-level quantisation (Section 5, INT8 evaluation): the tensor is replaced by the
 * values its int8 codes stand for.  code = clamp(rint(x / scale), -127, 127), ties to even,
 * everything in fp64; y = code * scale.  codes may be NULL. */
void nmo_fake_quant(const double* x, int64_t count, double scale, double* y, int8_t* codes)
{
    for (int64_t i = 0; i < count; ++i) {
        double r = rint(x[i] / scale);
        if (r > 127.0) r = 127.0;
        if (r < -127.0) r = -127.0;
        if (codes) codes[i] = (int8_t)r;
        y[i] = r * scale;
    }
}

/* ---- CNN pieces (NHWC) -------------------------------------------------------- */

/* out[n][oy][ox][co] = PWL( sum_{ky,kx,ci} in[n][oy*s-p+ky][ox*s-p+kx][ci] * W[co][ky][kx][ci]
 *                           + bias[co] ) + residual[n][oy][ox][co]
 * zero padding; W is [Cout, kh, kw, Cin]. */
void nmo_conv2d_nhwc(const double* in, int32_t Nb, int32_t Hin, int32_t Win, int32_t Cin,
                     const double* W, int32_t Cout, int32_t kh, int32_t kw,
                     int32_t stride, int32_t pad, const double* bias, const double* residual,
                     const nmo_pwl* t, double* out)
{
    int32_t Ho = (Hin + 2 * pad - kh) / stride + 1;
    int32_t Wo = (Win + 2 * pad - kw) / stride + 1;
    int64_t rows = (int64_t)Nb * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        int32_t n = (int32_t)(r / ((int64_t)Ho * Wo));
        int32_t oy = (int32_t)((r / Wo) % Ho);
        int32_t ox = (int32_t)(r % Wo);
        for (int32_t co = 0; co < Cout; ++co) {
            double acc = 0.0;
            for (int32_t ky = 0; ky < kh; ++ky) {
                int32_t iy = oy * stride - pad + ky;
                if (iy < 0 || iy >= Hin) continue;
                for (int32_t kx = 0; kx < kw; ++kx) {
                    int32_t ix = ox * stride - pad + kx;
                    if (ix < 0 || ix >= Win) continue;
                    const double* ip = in + (((int64_t)n * Hin + iy) * Win + ix) * Cin;
                    const double* wp = W + (((int64_t)co * kh + ky) * kw + kx) * Cin;
                    for (int32_t ci = 0; ci < Cin; ++ci) acc += ip[ci] * wp[ci];
                }
            }
            if (bias) acc += bias[co];
            if (t) acc = pwl_one(t, acc, NULL);
            if (residual) acc += residual[r * Cout + co];
            out[r * Cout + co] = acc;
        }
    }
}

/* window maximum, padding cells ignored */
void nmo_maxpool_nhwc(const double* in, int32_t Nb, int32_t Hin, int32_t Win, int32_t C,
                      int32_t ksz, int32_t stride, int32_t pad, double* out)
{
    int32_t Ho = (Hin + 2 * pad - ksz) / stride + 1;
    int32_t Wo = (Win + 2 * pad - ksz) / stride + 1;
    for (int32_t n = 0; n < Nb; ++n)
        for (int32_t oy = 0; oy < Ho; ++oy)
            for (int32_t ox = 0; ox < Wo; ++ox)
                for (int32_t c = 0; c < C; ++c) {
                    double m = -INFINITY;
                    for (int32_t ky = 0; ky < ksz; ++ky)
                        for (int32_t kx = 0; kx < ksz; ++kx) {
                            int32_t iy = oy * stride - pad + ky, ix = ox * stride - pad + kx;
                            if (iy < 0 || iy >= Hin || ix < 0 || ix >= Win) continue;
                            double v = in[(((int64_t)n * Hin + iy) * Win + ix) * C + c];
                            if (v > m) m = v;
                        }
                    out[(((int64_t)n * Ho + oy) * Wo + ox) * C + c] = m;
                }
}

/* mean over all spatial positions: [N,H,W,C] -> [N,C] */
void nmo_avgpool_nhwc(const double* in, int32_t Nb, int32_t Hin, int32_t Win, int32_t C, double* out)
{
    for (int32_t n = 0; n < Nb; ++n)
        for (int32_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int64_t p = 0; p < (int64_t)Hin * Win; ++p) s += in[((int64_t)n * Hin * Win + p) * C + c];
            out[(int64_t)n * C + c] = s / (double)((int64_t)Hin * Win);
        }
}
