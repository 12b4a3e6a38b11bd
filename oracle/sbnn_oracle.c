/*
 * CPU oracle for group-sparse convolution.  TEST INFRASTRUCTURE ONLY.
 *
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
 * call this file.  It shares no code with the CUDA library and the library
 * never calls it.
 *
 * What it computes: the sparse engine's result is, by definition, an ordinary
 * convolution with the masked weight  W~ = W (.) M  (paper Section 3.1).  So
 * the oracle is that definition written out: a dense direct convolution that
 * multiplies every weight by its 0/1 mask entry, visits every input channel
 * (no zero skipping, no packed format), and accumulates in double precision in
 * the natural loop order.  Tensors follow Algorithm 1's shapes: activations
 * [n][h][w][c], weights [oc][kh][kw][ic].  Zero padding (K-1)/2, cross-
 * correlation, bias added before the optional ReLU.
 *
 * Besides the result each routine returns, per output, S = |b| + sum |w*m*x|,
 * the scale against which a floating-point implementation is compared.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* fp32 -> bf16 -> fp32, round to nearest even (bf16 keeps the top 16 bits of an IEEE-754 binary32). */
static float bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return f; /* inf / nan unchanged */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

void oracle_bf16_round(const float* in, float* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_rne(in[i]);
}

/*
 * Dense direct convolution over masked weights.
 *   X    [N][H][Wd][Cin]           W, M [Cout][KH][KW][Cin]      bias [Cout] or NULL
 *   ref, S [N][Ho][Wo][Cout] (double), Ho = (H + 2*ph - KH)/stride + 1, ph = (KH-1)/2
 * round_bf16 != 0: w*m and x are rounded to bf16 before they are multiplied.
 */
void oracle_conv2d(const float* X, const float* W, const uint8_t* M, const float* bias,
                   int N, int H, int Wd, int Cin, int Cout, int KH, int KW, int stride,
                   int relu, int round_bf16, double* ref, double* S) {
    const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
    const int Ho = (H + 2 * ph - KH) / stride + 1;
    const int Wo = (Wd + 2 * pw - KW) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox)
                for (int o = 0; o < Cout; ++o) {
                    double b = bias ? (double)bias[o] : 0.0;
                    double acc = b, s = fabs(b);
                    for (int kh = 0; kh < KH; ++kh) {
                        int iy = oy * stride + kh - ph;
                        if (iy < 0 || iy >= H) continue;
                        for (int kw = 0; kw < KW; ++kw) {
                            int ix = ox * stride + kw - pw;
                            if (ix < 0 || ix >= Wd) continue;
                            const float* xp = X + (((int64_t)n * H + iy) * Wd + ix) * Cin;
                            const int64_t wo = (((int64_t)o * KH + kh) * KW + kw) * Cin;
                            for (int c = 0; c < Cin; ++c) {
                                float wm = M[wo + c] ? W[wo + c] : 0.0f;
                                float xv = xp[c];
                                if (round_bf16) { wm = bf16_rne(wm); xv = bf16_rne(xv); }
                                double p = (double)wm * (double)xv;
                                acc += p;
                                s += fabs(p);
                            }
                        }
                    }
                    int64_t oi = (((int64_t)n * Ho + oy) * Wo + ox) * Cout + o;
                    ref[oi] = (relu && acc < 0.0) ? 0.0 : acc;
                    S[oi] = s;
                }
}

/*
 * Dense depthwise 3x3, pad 1.  X [N][H][Wd][C], W [3][3][C], bias [C] or NULL,
 * ref, S [N][Ho][Wo][C] with Ho = (H - 1)/stride + 1.
 */
void oracle_dwconv3x3(const float* X, const float* W, const float* bias, int N, int H, int Wd, int C,
                      int stride, int relu, double* ref, double* S) {
    const int Ho = (H + 2 - 3) / stride + 1, Wo = (Wd + 2 - 3) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox)
                for (int c = 0; c < C; ++c) {
                    double b = bias ? (double)bias[c] : 0.0;
                    double acc = b, s = fabs(b);
                    for (int kh = 0; kh < 3; ++kh) {
                        int iy = oy * stride + kh - 1;
                        if (iy < 0 || iy >= H) continue;
                        for (int kw = 0; kw < 3; ++kw) {
                            int ix = ox * stride + kw - 1;
                            if (ix < 0 || ix >= Wd) continue;
                            double p = (double)W[(kh * 3 + kw) * C + c] *
                                       (double)X[(((int64_t)n * H + iy) * Wd + ix) * C + c];
                            acc += p;
                            s += fabs(p);
                        }
                    }
                    int64_t oi = (((int64_t)n * Ho + oy) * Wo + ox) * C + c;
                    ref[oi] = (relu && acc < 0.0) ? 0.0 : acc;
                    S[oi] = s;
                }
}

/* Mean over the HW positions of every (image, channel).  X [N][HW][C] -> ref, S [N][C]; S = mean |x|. */
void oracle_avgpool(const float* X, int N, int HW, int C, double* ref, double* S) {
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            double acc = 0.0, s = 0.0;
            for (int p = 0; p < HW; ++p) {
                double v = (double)X[((int64_t)n * HW + p) * C + c];
                acc += v;
                s += fabs(v);
            }
            ref[(int64_t)n * C + c] = acc / HW;
            S[(int64_t)n * C + c] = s / HW;
        }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
