/*
 * gf_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the filtered convolution backward
 * pass of gradient filtering (Yang, Li, Marculescu, CVPR 2023) computes.
 * Everything is a direct loop nest over the paper's indices; there is no
 * blocking, fusion or reordering.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call into this file.  It shares no code with
 * the CUDA library and includes none of its headers.
 *
 * Notation (paper, Table of symbols): x[n,c_i,h,w], theta[c_o,c_i,u,v], g_y,
 * g_x, g_theta, patch size r.  All tensors are dense, row-major, NCHW / OIHW.
 * Grouped convolutions: theta is [C_out, C_in/G, KH, KW]; output channel c_o
 * belongs to group q = c_o / (C_out/G) and sees input channels
 * q*C_in/G ... (q+1)*C_in/G - 1.
 *
 * Readings taken where the paper's text is garbled or silent:
 *   - Patch (a,b) of an H x W map is the half-open index block
 *     [a r, min((a+1) r, H)) x [b r, min((b+1) r, W)); there are
 *     ceil(H/r) x ceil(W/r) patches (Section 3.3: the prose describes the map
 *     as tiled by r x r blocks, and the count of unique values is stated right
 *     after the filter equation).  The printed summation limits are not used.
 *   - On a partial patch at the right/bottom edge the patch value is the
 *     mean over the elements that exist.  PARITY UNPINNED for this divisor:
 *     the paper gives no worked example with a partial patch (its formula
 *     prints 1/r^2, its prose speaks of an average).
 *   - Eq. (grad_w) is summed once per patch: sum_{n,a,b} xsum * gmean, which
 *     is what the first line of its derivation in the supplement gives at
 *     zero offset without any approximation.
 *   - r == 1 means the method is off: exact convolution backward (Section
 *     4.2 names the 1 x 1 patch size as its exact-backpropagation baseline).
 *   - Stride 1, dilation 1, odd kernels with pad = (K-1)/2, the geometry in
 *     which Eq. (grad_x) indexes g_x and g_y with the same (h,w).
 */
#include <stddef.h>
#include <stdint.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static int64_t imin(int64_t a, int64_t b) { return a < b ? a : b; }

int gfo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Section 3.4, text after Eq. (grad_w); supplement "Approximation for Input
 * Feature x": xs[n,c,a,b] = sum of x over patch (a,b). */
void gfo_patch_sum(const double* x, int64_t N, int64_t C, int64_t H, int64_t W,
                   int64_t r, double* xs) {
    const int64_t Hp = cdiv(H, r), Wp = cdiv(W, r);
#pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc) {
        const double* plane = x + nc * H * W;
        for (int64_t a = 0; a < Hp; ++a)
            for (int64_t b = 0; b < Wp; ++b) {
                double s = 0.0;
                for (int64_t i = a * r; i < imin((a + 1) * r, H); ++i)
                    for (int64_t j = b * r; j < imin((b + 1) * r, W); ++j)
                        s += plane[i * W + j];
                xs[(nc * Hp + a) * Wp + b] = s;
            }
    }
}

/* Section 3.3 (gradient filter): the unique-value matrix of g~_y,
 * gm[n,c,a,b] = average of g_y over patch (a,b). */
void gfo_patch_mean(const double* g, int64_t N, int64_t C, int64_t H, int64_t W,
                    int64_t r, double* gm) {
    const int64_t Hp = cdiv(H, r), Wp = cdiv(W, r);
#pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc) {
        const double* plane = g + nc * H * W;
        for (int64_t a = 0; a < Hp; ++a)
            for (int64_t b = 0; b < Wp; ++b) {
                double s = 0.0;
                int64_t cnt = 0;
                for (int64_t i = a * r; i < imin((a + 1) * r, H); ++i)
                    for (int64_t j = b * r; j < imin((b + 1) * r, W); ++j) {
                        s += plane[i * W + j];
                        ++cnt;
                    }
                gm[(nc * Hp + a) * Wp + b] = s / (double)cnt;
            }
    }
}

/* Supplement "Gradient Filtering": unique values back to full resolution,
 * full[n,c,h,w] = u[n,c,floor(h/r),floor(w/r)]. */
void gfo_expand(const double* u, int64_t N, int64_t C, int64_t H, int64_t W,
                int64_t r, double* full) {
    const int64_t Hp = cdiv(H, r), Wp = cdiv(W, r);
#pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc)
        for (int64_t h = 0; h < H; ++h)
            for (int64_t w = 0; w < W; ++w)
                full[(nc * H + h) * W + w] = u[(nc * Hp + h / r) * Wp + w / r];
}

/* Text under Eq. (grad_x); supplement "Approximation for Rotated Convolution
 * Kernel": ts[c_o,c_l] = sum_{u,v} theta[c_o,c_l,u,v] (rot180 drops out). */
void gfo_kernel_sum(const double* theta, int64_t Cout, int64_t Cig, int64_t KH,
                    int64_t KW, double* ts) {
    for (int64_t oc = 0; oc < Cout * Cig; ++oc) {
        double s = 0.0;
        for (int64_t t = 0; t < KH * KW; ++t) s += theta[oc * KH * KW + t];
        ts[oc] = s;
    }
}

/* Eq. (grad_w), summed once per patch, written to every tap (u,v):
 * gw[c_o,c_l,u,v] = sum_{n,a,b} xs[n, q C_ig + c_l, a, b] * gm[n, c_o, a, b]. */
void gfo_reduced_gw(const double* xs, const double* gm, int64_t N, int64_t Cin,
                    int64_t Cout, int64_t G, int64_t Hp, int64_t Wp, int64_t KH,
                    int64_t KW, double* gw) {
    const int64_t Cig = Cin / G, Cog = Cout / G, P = Hp * Wp;
#pragma omp parallel for schedule(static)
    for (int64_t co = 0; co < Cout; ++co) {
        const int64_t q = co / Cog;
        for (int64_t cl = 0; cl < Cig; ++cl) {
            const int64_t ci = q * Cig + cl;
            double s = 0.0;
            for (int64_t n = 0; n < N; ++n)
                for (int64_t p = 0; p < P; ++p)
                    s += xs[(n * Cin + ci) * P + p] * gm[(n * Cout + co) * P + p];
            for (int64_t t = 0; t < KH * KW; ++t)
                gw[(co * Cig + cl) * KH * KW + t] = s;
        }
    }
}

/* Eq. (grad_x) with the expansion of the supplement's Eq. (gx_final):
 * gx[n,c_i,h,w] = sum_{c_o in group(c_i)} gm[n,c_o,floor(h/r),floor(w/r)]
 *                                        * ts[c_o, c_i - q C_ig]. */
void gfo_reduced_gx(const double* gm, const double* ts, int64_t N, int64_t Cin,
                    int64_t Cout, int64_t G, int64_t H, int64_t W, int64_t r,
                    double* gx) {
    const int64_t Cig = Cin / G, Cog = Cout / G;
    const int64_t Hp = cdiv(H, r), Wp = cdiv(W, r);
#pragma omp parallel for schedule(static)
    for (int64_t nci = 0; nci < N * Cin; ++nci) {
        const int64_t n = nci / Cin, ci = nci % Cin;
        const int64_t q = ci / Cig, cl = ci % Cig;
        for (int64_t h = 0; h < H; ++h)
            for (int64_t w = 0; w < W; ++w) {
                double s = 0.0;
                for (int64_t co = q * Cog; co < (q + 1) * Cog; ++co)
                    s += gm[((n * Cout + co) * Hp + h / r) * Wp + w / r] *
                         ts[co * Cig + cl];
                gx[(nci * H + h) * W + w] = s;
            }
    }
}

/* Section 3.1: exact ("vanilla") convolution backward by brute force, stride 1,
 * zero padding (ph, pw); output map size Hy = H + 2 ph - KH + 1 (same for W).
 *   g_theta[c_o,c_l,u,v] = sum_{n,i,j} x[n,c_i,i+u-ph,j+v-pw] g_y[n,c_o,i,j]
 *   g_x = g_y (*) rot180(theta), i.e.
 *   g_x[n,c_i,h,w] = sum_{c_o,u,v} theta[c_o,c_l,u,v] g_y[n,c_o,h-u+ph,w-v+pw]
 * with out-of-range reads equal to zero.  Either output may be NULL. */
void gfo_exact_backward(const double* x, const double* gy, const double* theta,
                        int64_t N, int64_t Cin, int64_t Cout, int64_t G,
                        int64_t H, int64_t W, int64_t KH, int64_t KW, int64_t ph,
                        int64_t pw, double* gw, double* gx) {
    const int64_t Cig = Cin / G, Cog = Cout / G;
    const int64_t Hy = H + 2 * ph - KH + 1, Wy = W + 2 * pw - KW + 1;
    if (gw) {
#pragma omp parallel for schedule(static)
        for (int64_t co = 0; co < Cout; ++co) {
            const int64_t q = co / Cog;
            for (int64_t cl = 0; cl < Cig; ++cl) {
                const int64_t ci = q * Cig + cl;
                for (int64_t u = 0; u < KH; ++u)
                    for (int64_t v = 0; v < KW; ++v) {
                        double s = 0.0;
                        for (int64_t n = 0; n < N; ++n)
                            for (int64_t i = 0; i < Hy; ++i)
                                for (int64_t j = 0; j < Wy; ++j) {
                                    const int64_t h = i + u - ph, w = j + v - pw;
                                    if (h < 0 || h >= H || w < 0 || w >= W) continue;
                                    s += x[((n * Cin + ci) * H + h) * W + w] *
                                         gy[((n * Cout + co) * Hy + i) * Wy + j];
                                }
                        gw[((co * Cig + cl) * KH + u) * KW + v] = s;
                    }
            }
        }
    }
    if (gx) {
#pragma omp parallel for schedule(static)
        for (int64_t nci = 0; nci < N * Cin; ++nci) {
            const int64_t n = nci / Cin, ci = nci % Cin;
            const int64_t q = ci / Cig, cl = ci % Cig;
            for (int64_t h = 0; h < H; ++h)
                for (int64_t w = 0; w < W; ++w) {
                    double s = 0.0;
                    for (int64_t co = q * Cog; co < (q + 1) * Cog; ++co)
                        for (int64_t u = 0; u < KH; ++u)
                            for (int64_t v = 0; v < KW; ++v) {
                                const int64_t i = h - u + ph, j = w - v + pw;
                                if (i < 0 || i >= Hy || j < 0 || j >= Wy) continue;
                                s += theta[((co * Cig + cl) * KH + u) * KW + v] *
                                     gy[((n * Cout + co) * Hy + i) * Wy + j];
                            }
                    gx[(nci * H + h) * W + w] = s;
                }
        }
    }
}

/* Supplement "Boundary Elements": a patch-constant field extended ("padded")
 * to every integer offset (i,j) around its own patch -- whatever the offset,
 * the value is the patch's unique value. */
static double padded_patch(const double* uniq, int64_t plane, int64_t Hp,
                           int64_t Wp, int64_t hp, int64_t wp, int64_t i,
                           int64_t j) {
    (void)i;
    (void)j;
    return uniq[(plane * Hp + hp) * Wp + wp];
}

/* The derivations of the supplement taken literally, for "same" geometry
 * (odd K, pad (K-1)/2, stride 1): exact backward written with centred kernel
 * offsets, in which every read of g~_y (for g_x) or of the approximated x (for
 * g_theta) that the kernel makes around pixel (h,w) is served by the padded
 * patch that contains (h,w).  theta is NOT pre-summed and nothing is summed per
 * patch: the loops run over full-resolution pixels and kernel taps.
 *   gm    : unique values of g~_y                       [N,Cout,Hp,Wp]
 *   xmean : x replaced by a patch-constant field whose unique value is
 *           xs / |patch| (so that a sum over the patch's pixels gives xs) [N,Cin,Hp,Wp]
 */
void gfo_literal_backward(const double* xmean, const double* gm,
                          const double* theta, int64_t N, int64_t Cin,
                          int64_t Cout, int64_t G, int64_t H, int64_t W,
                          int64_t r, int64_t KH, int64_t KW, double* gw,
                          double* gx) {
    const int64_t Cig = Cin / G, Cog = Cout / G;
    const int64_t Hp = cdiv(H, r), Wp = cdiv(W, r);
    const int64_t ch = (KH - 1) / 2, cw = (KW - 1) / 2;
    if (gx) {
#pragma omp parallel for schedule(static)
        for (int64_t nci = 0; nci < N * Cin; ++nci) {
            const int64_t n = nci / Cin, ci = nci % Cin;
            const int64_t q = ci / Cig, cl = ci % Cig;
            for (int64_t h = 0; h < H; ++h)
                for (int64_t w = 0; w < W; ++w) {
                    double s = 0.0;
                    for (int64_t co = q * Cog; co < (q + 1) * Cog; ++co)
                        for (int64_t u = -ch; u <= ch; ++u)
                            for (int64_t v = -cw; v <= cw; ++v)
                                /* theta[c_o,c_i,-u,-v] in centred offsets */
                                s += theta[((co * Cig + cl) * KH + (ch - u)) * KW + (cw - v)] *
                                     padded_patch(gm, n * Cout + co, Hp, Wp, h / r,
                                                  w / r, h % r + u, w % r + v);
                    gx[(nci * H + h) * W + w] = s;
                }
        }
    }
    if (gw) {
#pragma omp parallel for schedule(static)
        for (int64_t co = 0; co < Cout; ++co) {
            const int64_t q = co / Cog;
            for (int64_t cl = 0; cl < Cig; ++cl) {
                const int64_t ci = q * Cig + cl;
                for (int64_t u = -ch; u <= ch; ++u)
                    for (int64_t v = -cw; v <= cw; ++v) {
                        double s = 0.0;
                        for (int64_t n = 0; n < N; ++n)
                            for (int64_t h = 0; h < H; ++h)
                                for (int64_t w = 0; w < W; ++w)
                                    s += padded_patch(xmean, n * Cin + ci, Hp, Wp,
                                                      h / r, w / r, h % r + u,
                                                      w % r + v) *
                                         padded_patch(gm, n * Cout + co, Hp, Wp,
                                                      h / r, w / r, h % r, w % r);
                        gw[((co * Cig + cl) * KH + (u + ch)) * KW + (v + cw)] = s;
                    }
            }
        }
    }
}
