/* CPU oracle for the floating-point part of the path: what every source token
 * gets back from this GPU's local experts, and their gate-weighted sum.
 *
 * TEST INFRASTRUCTURE ONLY.  The product path never links, loads or calls this
 * file; tests, the smoke check and the benchmark's CPU-baseline leg do.  It
 * shares no code, header, table or helper with the CUDA path.
 *
 * The method reorders and overlaps work but reaches exactly the plain MoE
 * result (Section 2.1: the layer output is the gate-weighted sum of the selected
 * experts' outputs; steps 3-5 of the forward pass), so this is that definition
 * written out as a per-token loop over the token's top-k experts, restricted to
 * the experts held locally, in ascending expert index:
 *
 *   gq_j = sum_c x[c] * W1[e][j][c]         up_j = sum_c x[c] * W1[e][F+j][c]
 *   h_j  = bf16( gq_j / (1 + exp(-gq_j)) * up_j )           (SwiGLU, fp32 math)
 *   y_c  = bf16( sum_j h_j * W2[e][c][j] )                  (expert output row)
 *   acc_c += gate_e * float(y_c)                            (step 5, at the owner)
 *   out_c = bf16(acc_c); a token with no local expert gets +0
 *
 * Accumulation is fp32 throughout; values are rounded to bf16 (round to nearest
 * even) exactly where the path has to materialise bf16: the hidden row h, the
 * returned row y, and the final output.  Gates are used as given; y is returned
 * unscaled because the scaling happens at the owner rank.
 *
 * moe_oracle_tokens_single is the same for experts that are one projection each
 * (the operator of the paper's Table 2).
 *
 * Pins (tests/test_oracle_values.py): float64 NumPy evaluation of the
 * definition on tiny inputs, a one-expert case against library matmul/silu,
 * zero gate projection => exact zeros, identity experts with unit gates
 * reproducing x bit-exactly, and gate linearity.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static float bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static uint16_t f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u)      /* NaN stays NaN */
        return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7fffu + ((u >> 16) & 1u);          /* round to nearest even */
    return (uint16_t)(u >> 16);
}

/* One expert applied to one token row.  xf: d floats; hf: F floats of scratch;
 * y: d bf16 values out. */
static void expert_ffn(const float *xf, const uint16_t *w1, const uint16_t *w2, int d, int F,
                       float *hf, uint16_t *y)
{
    for (int j = 0; j < F; ++j) {
        const uint16_t *wg = w1 + (size_t)j * d;
        const uint16_t *wu = w1 + (size_t)(F + j) * d;
        float gq = 0.0f, up = 0.0f;
        for (int c = 0; c < d; ++c) {
            gq += xf[c] * bf16_to_f32(wg[c]);
            up += xf[c] * bf16_to_f32(wu[c]);
        }
        float h = gq / (1.0f + expf(-gq)) * up;
        hf[j] = bf16_to_f32(f32_to_bf16(h));
    }
    for (int c = 0; c < d; ++c) {
        const uint16_t *w = w2 + (size_t)c * F;
        float s = 0.0f;
        for (int j = 0; j < F; ++j)
            s += hf[j] * bf16_to_f32(w[j]);
        y[c] = f32_to_bf16(s);
    }
}

/* Evaluates n_sel tokens (flat index r*T + t into x / expert / gate).
 *   x      [R*T, d] bf16      expert [R*T, k] global expert ids      gate [R*T, k] fp32
 *   w1     [El, 2F, d] bf16   w2     [El, d, F] bf16   (local experts = global ids first_local..+El-1)
 *   out    [n_sel, d] bf16
 *   y      [n_sel, kmax, d] bf16, j-th local expert of the token in ascending expert order (zeros if none)
 *   y_exp  [n_sel, kmax] local expert index of that row, or -1
 * Returns 0, or -1 if a token selects more than kmax local experts. */
int moe_oracle_tokens(int T, int k, int d, int F, int El, int first_local,
                      const uint16_t *x, const int32_t *expert, const float *gate,
                      const uint16_t *w1, const uint16_t *w2,
                      int n_sel, const int32_t *sel, int kmax,
                      uint16_t *out, uint16_t *y, int32_t *y_exp, int nthreads)
{
    int bad = 0;
    (void)T;
#ifdef _OPENMP
    if (nthreads > 0)
        omp_set_num_threads(nthreads);
#endif
#pragma omp parallel
    {
        float *xf = (float *)malloc(sizeof(float) * (size_t)d);
        float *hf = (float *)malloc(sizeof(float) * (size_t)F);
        float *acc = (float *)malloc(sizeof(float) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int s = 0; s < n_sel; ++s) {
            const int tok = sel[s];
            const uint16_t *xr = x + (size_t)tok * d;
            for (int c = 0; c < d; ++c) {
                xf[c] = bf16_to_f32(xr[c]);
                acc[c] = 0.0f;
            }
            int nloc = 0;
            for (int j = 0; j < kmax; ++j) {
                y_exp[(size_t)s * kmax + j] = -1;
                memset(y + ((size_t)s * kmax + j) * d, 0, sizeof(uint16_t) * (size_t)d);
            }
            /* the token's selected experts that live here, ascending expert index */
            for (int e = 0; e < El; ++e) {
                int hit = -1;
                for (int q = 0; q < k; ++q)
                    if (expert[(size_t)tok * k + q] == first_local + e)
                        hit = q;
                if (hit < 0)
                    continue;
                if (nloc >= kmax) {
                    bad = 1;
                    break;
                }
                uint16_t *yr = y + ((size_t)s * kmax + nloc) * d;
                expert_ffn(xf, w1 + (size_t)e * 2 * F * d, w2 + (size_t)e * d * F, d, F, hf, yr);
                const float g = gate[(size_t)tok * k + hit];
                for (int c = 0; c < d; ++c)
                    acc[c] += g * bf16_to_f32(yr[c]);
                y_exp[(size_t)s * kmax + nloc] = e;
                ++nloc;
            }
            for (int c = 0; c < d; ++c)
                out[(size_t)s * d + c] = f32_to_bf16(acc[c]);
        }
        free(xf);
        free(hf);
        free(acc);
    }
    return bad ? -1 : 0;
}

/* The operator the paper evaluates (Table 2: one M x K x N GEMM per expert, "the expert output projection"):
 * each expert is a single projection, y_j = bf16( sum_c x[c] * W[e][j][c] ), j = 0..N-1, followed by the same
 * gate-weighted sum at the owner.  Same arguments as moe_oracle_tokens with w [El, N, d]; out [n_sel, N],
 * y [n_sel, kmax, N]. */
int moe_oracle_tokens_single(int T, int k, int d, int N, int El, int first_local,
                             const uint16_t *x, const int32_t *expert, const float *gate, const uint16_t *w,
                             int n_sel, const int32_t *sel, int kmax,
                             uint16_t *out, uint16_t *y, int32_t *y_exp, int nthreads)
{
    int bad = 0;
    (void)T;
#ifdef _OPENMP
    if (nthreads > 0)
        omp_set_num_threads(nthreads);
#endif
#pragma omp parallel
    {
        float *xf = (float *)malloc(sizeof(float) * (size_t)d);
        float *acc = (float *)malloc(sizeof(float) * (size_t)N);
#pragma omp for schedule(dynamic, 1)
        for (int s = 0; s < n_sel; ++s) {
            const int tok = sel[s];
            for (int c = 0; c < d; ++c)
                xf[c] = bf16_to_f32(x[(size_t)tok * d + c]);
            for (int j = 0; j < N; ++j)
                acc[j] = 0.0f;
            int nloc = 0;
            for (int j = 0; j < kmax; ++j) {
                y_exp[(size_t)s * kmax + j] = -1;
                memset(y + ((size_t)s * kmax + j) * N, 0, sizeof(uint16_t) * (size_t)N);
            }
            for (int e = 0; e < El; ++e) {
                int hit = -1;
                for (int q = 0; q < k; ++q)
                    if (expert[(size_t)tok * k + q] == first_local + e)
                        hit = q;
                if (hit < 0)
                    continue;
                if (nloc >= kmax) {
                    bad = 1;
                    break;
                }
                uint16_t *yr = y + ((size_t)s * kmax + nloc) * N;
                const float g = gate[(size_t)tok * k + hit];
                for (int j = 0; j < N; ++j) {
                    const uint16_t *wr = w + ((size_t)e * N + j) * d;
                    float v = 0.0f;
                    for (int c = 0; c < d; ++c)
                        v += xf[c] * bf16_to_f32(wr[c]);
                    yr[j] = f32_to_bf16(v);
                    acc[j] += g * bf16_to_f32(yr[j]);
                }
                y_exp[(size_t)s * kmax + nloc] = e;
                ++nloc;
            }
            for (int j = 0; j < N; ++j)
                out[(size_t)s * N + j] = f32_to_bf16(acc[j]);
        }
        free(xf);
        free(acc);
    }
    return bad ? -1 : 0;
}

int moe_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
