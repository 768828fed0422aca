/*
 * TEST INFRASTRUCTURE ONLY -- the fp64 CPU oracle for the AlexNet training step.
 *
 * Plain definitions of every layer's forward and analytic backward, in double
 * precision, canonical NCHW / OIHW layouts, naive loops.  Nothing here is
 * blocked, fused or reordered beyond what the definitions state (OpenMP only
 * spreads independent output planes over cores).  It shares no code, header,
 * table or layout with the CUDA path and must never be called from it; only
 * the tests, the smoke check and the bench's cpu-baseline leg load this file.
 *
 * What each function follows:
 *   - topology (5 conv, 3 max-pool, 2 FC, softmax): the paper's Methods section;
 *     all layer constants are those of Krizhevsky et al. 2012, which it cites.
 *   - preprocessing (mean-image subtract, random crop, random flip): the
 *     footnote of the "Parallel Data Loading" subsection.
 *   - exchange-and-average of weights, biases and momentum: the "Data
 *     parallelism" subsection and its figure (done in numpy by the caller).
 *
 * Parity status: every function below is pinned by tests/test_oracle_*.py
 * (closed forms, brute force, finite differences, library special cases).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

/* ---------------------------------------------------------------- hashing */
/* Counter-based generator: the 64-bit finaliser of SplitMix64 (Steele, Lea,
 * Flood 2014) applied to key + golden*(idx+1).  Pure integer arithmetic, so
 * any two implementations agree bit for bit. */
uint64_t orc_mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}
uint64_t orc_key(uint64_t seed, uint64_t stream, uint64_t replica, uint64_t step) {
    return orc_mix64(seed ^ (stream << 56) ^ (replica << 48) ^ step);
}
uint64_t orc_draw(uint64_t key, uint64_t idx) {
    return orc_mix64(key + 0x9E3779B97F4A7C15ULL * (idx + 1));
}

/* crop offsets and flip bit per image: stream 1, idx = image number.
 * out[n] = (ox, oy, flip), ox,oy in [0,29]. */
void orc_crop_flip(uint64_t seed, uint64_t replica, uint64_t step, int B, int32_t* out) {
    uint64_t key = orc_key(seed, 1, replica, step);
    for (int n = 0; n < B; ++n) {
        uint64_t r = orc_draw(key, (uint64_t)n);
        out[3 * n + 0] = (int32_t)((r & 0xFFFF) % 30);
        out[3 * n + 1] = (int32_t)(((r >> 16) & 0xFFFF) % 30);
        out[3 * n + 2] = (int32_t)((r >> 32) & 1);
    }
}

/* dropout keep-mask: stream 2 (fc6) or 3 (fc7), idx = n*width + j;
 * keep iff the top 24 bits of the draw are >= floor(p * 2^24). */
void orc_dropout_mask(uint64_t seed, uint64_t stream, uint64_t replica, uint64_t step,
                      int B, int width, double p, uint8_t* keep) {
    uint64_t key = orc_key(seed, stream, replica, step);
    uint64_t thr = (uint64_t)floor(p * 16777216.0);
    for (int64_t i = 0; i < (int64_t)B * width; ++i)
        keep[i] = ((orc_draw(key, (uint64_t)i) >> 40) >= thr) ? 1 : 0;
}

/* ---------------------------------------------------------- preprocessing */
/* X[n][c][y][x] = u8[n][sy][sx][c] - mean[sy][sx][c] with sy = oy + y and
 * sx = ox + (flip ? 226 - x : x): the mean image is taken at the source pixel
 * (subtract first, then crop, then flip). */
void orc_preprocess(const uint8_t* img, const double* mean, const int32_t* cf, int B, double* X) {
    #pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        int ox = cf[3 * n], oy = cf[3 * n + 1], flip = cf[3 * n + 2];
        for (int c = 0; c < 3; ++c)
            for (int y = 0; y < 227; ++y)
                for (int x = 0; x < 227; ++x) {
                    int sy = oy + y;
                    int sx = ox + (flip ? 226 - x : x);
                    size_t s = ((size_t)sy * 256 + sx) * 3 + c;
                    X[(((size_t)n * 3 + c) * 227 + y) * 227 + x] =
                        (double)img[(size_t)n * 256 * 256 * 3 + s] - mean[s];
                }
    }
}

/* ------------------------------------------------------------ convolution */
/* Cross-correlation (no kernel flip), groups: output channel co belongs to
 * group co / (Cout/G) and reads input channels [grp*Cin/G, (grp+1)*Cin/G).
 * y[n][co][oy][ox] = b[co] + sum_{ci',ky,kx} w[co][ci'][ky][kx] *
 *                    x[n][grp*Cin/G+ci'][oy*s+ky-p][ox*s+kx-p]   (zero outside) */
static int out_dim(int in, int k, int s, int p) { return (in + 2 * p - k) / s + 1; }

void orc_conv_fwd(const double* x, const double* w, const double* b, double* y,
                  int N, int Cin, int H, int W, int Cout, int kh, int kw, int s, int p, int G) {
    int Ho = out_dim(H, kh, s, p), Wo = out_dim(W, kw, s, p);
    int cig = Cin / G, cog = Cout / G;
    #pragma omp parallel for collapse(2)
    for (int n = 0; n < N; ++n)
        for (int co = 0; co < Cout; ++co) {
            double* yp = y + ((size_t)n * Cout + co) * Ho * Wo;
            for (int i = 0; i < Ho * Wo; ++i) yp[i] = b ? b[co] : 0.0;
            int grp = co / cog;
            for (int ci = 0; ci < cig; ++ci) {
                const double* xp = x + ((size_t)n * Cin + grp * cig + ci) * H * W;
                for (int ky = 0; ky < kh; ++ky)
                    for (int kx = 0; kx < kw; ++kx) {
                        double wv = w[(((size_t)co * cig + ci) * kh + ky) * kw + kx];
                        for (int oy = 0; oy < Ho; ++oy) {
                            int iy = oy * s + ky - p;
                            if (iy < 0 || iy >= H) continue;
                            for (int ox = 0; ox < Wo; ++ox) {
                                int ix = ox * s + kx - p;
                                if (ix < 0 || ix >= W) continue;
                                yp[oy * Wo + ox] += wv * xp[iy * W + ix];
                            }
                        }
                    }
            }
        }
}

/* dx[n][ci][iy][ix] = sum over (co in group, ky, kx, oy, ox) with
 * iy = oy*s+ky-p, ix = ox*s+kx-p of dy[n][co][oy][ox] * w[co][ci'][ky][kx]. */
void orc_conv_bwd_data(const double* dy, const double* w, double* dx,
                       int N, int Cin, int H, int W, int Cout, int kh, int kw, int s, int p, int G) {
    int Ho = out_dim(H, kh, s, p), Wo = out_dim(W, kw, s, p);
    int cig = Cin / G, cog = Cout / G;
    #pragma omp parallel for collapse(2)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < Cin; ++c) {
            double* dxp = dx + ((size_t)n * Cin + c) * H * W;
            for (int i = 0; i < H * W; ++i) dxp[i] = 0.0;
            int grp = c / cig, ci = c % cig;
            for (int co = grp * cog; co < (grp + 1) * cog; ++co) {
                const double* dyp = dy + ((size_t)n * Cout + co) * Ho * Wo;
                for (int ky = 0; ky < kh; ++ky)
                    for (int kx = 0; kx < kw; ++kx) {
                        double wv = w[(((size_t)co * cig + ci) * kh + ky) * kw + kx];
                        for (int oy = 0; oy < Ho; ++oy) {
                            int iy = oy * s + ky - p;
                            if (iy < 0 || iy >= H) continue;
                            for (int ox = 0; ox < Wo; ++ox) {
                                int ix = ox * s + kx - p;
                                if (ix < 0 || ix >= W) continue;
                                dxp[iy * W + ix] += dyp[oy * Wo + ox] * wv;
                            }
                        }
                    }
            }
        }
}

/* dw[co][ci'][ky][kx] = sum_{n,oy,ox} dy[n][co][oy][ox] * x[n][grp*Cin/G+ci'][oy*s+ky-p][ox*s+kx-p]
 * db[co] = sum_{n,oy,ox} dy[n][co][oy][ox] */
void orc_conv_bwd_weight(const double* x, const double* dy, double* dw, double* db,
                         int N, int Cin, int H, int W, int Cout, int kh, int kw, int s, int p, int G) {
    int Ho = out_dim(H, kh, s, p), Wo = out_dim(W, kw, s, p);
    int cig = Cin / G, cog = Cout / G;
    #pragma omp parallel for
    for (int co = 0; co < Cout; ++co) {
        int grp = co / cog;
        double bs = 0.0;
        for (int n = 0; n < N; ++n) {
            const double* dyp = dy + ((size_t)n * Cout + co) * Ho * Wo;
            for (int i = 0; i < Ho * Wo; ++i) bs += dyp[i];
        }
        if (db) db[co] = bs;
        for (int ci = 0; ci < cig; ++ci)
            for (int ky = 0; ky < kh; ++ky)
                for (int kx = 0; kx < kw; ++kx) {
                    double acc = 0.0;
                    for (int n = 0; n < N; ++n) {
                        const double* dyp = dy + ((size_t)n * Cout + co) * Ho * Wo;
                        const double* xp = x + ((size_t)n * Cin + grp * cig + ci) * H * W;
                        for (int oy = 0; oy < Ho; ++oy) {
                            int iy = oy * s + ky - p;
                            if (iy < 0 || iy >= H) continue;
                            for (int ox = 0; ox < Wo; ++ox) {
                                int ix = ox * s + kx - p;
                                if (ix < 0 || ix >= W) continue;
                                acc += dyp[oy * Wo + ox] * xp[iy * W + ix];
                            }
                        }
                    }
                    dw[(((size_t)co * cig + ci) * kh + ky) * kw + kx] = acc;
                }
    }
}

/* ------------------------------------------------------------------- LRN */
/* Across-channel local response normalisation (Krizhevsky et al. 2012, Sec. 3.3):
 *   s_c = k + alpha * sum_{c' in [max(0,c-n/2), min(C-1,c+n/2)]} a_{c'}^2   (alpha NOT divided by n)
 *   b_c = a_c * s_c^(-beta) */
void orc_lrn_fwd(const double* a, double* b, double* scale_out /* may be NULL */,
                 int N, int C, int HW, int size, double alpha, double beta, double k) {
    int half = size / 2;
    #pragma omp parallel for
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            int lo = c - half < 0 ? 0 : c - half;
            int hi = c + half > C - 1 ? C - 1 : c + half;
            for (int i = 0; i < HW; ++i) {
                double ss = 0.0;
                for (int cc = lo; cc <= hi; ++cc) {
                    double v = a[((size_t)n * C + cc) * HW + i];
                    ss += v * v;
                }
                double sc = k + alpha * ss;
                size_t o = ((size_t)n * C + c) * HW + i;
                if (scale_out) scale_out[o] = sc;
                b[o] = a[o] * pow(sc, -beta);
            }
        }
}

/* da_m = g_m s_m^(-beta) - 2 alpha beta a_m sum_{c : m in window(c)} g_c a_c s_c^(-beta-1);
 * with a symmetric clipped window, {c : m in window(c)} = [m-n/2, m+n/2] clipped. */
void orc_lrn_bwd(const double* a, const double* g, double* da,
                 int N, int C, int HW, int size, double alpha, double beta, double k) {
    int half = size / 2;
    #pragma omp parallel for
    for (int n = 0; n < N; ++n)
        for (int i = 0; i < HW; ++i) {
            double s[1024];
            for (int c = 0; c < C; ++c) {
                int lo = c - half < 0 ? 0 : c - half;
                int hi = c + half > C - 1 ? C - 1 : c + half;
                double ss = 0.0;
                for (int cc = lo; cc <= hi; ++cc) {
                    double v = a[((size_t)n * C + cc) * HW + i];
                    ss += v * v;
                }
                s[c] = k + alpha * ss;
            }
            for (int m = 0; m < C; ++m) {
                int lo = m - half < 0 ? 0 : m - half;
                int hi = m + half > C - 1 ? C - 1 : m + half;
                double acc = 0.0;
                for (int c = lo; c <= hi; ++c) {
                    size_t o = ((size_t)n * C + c) * HW + i;
                    acc += g[o] * a[o] * pow(s[c], -beta - 1.0);
                }
                size_t om = ((size_t)n * C + m) * HW + i;
                da[om] = g[om] * pow(s[m], -beta) - 2.0 * alpha * beta * a[om] * acc;
            }
        }
}

/* -------------------------------------------------------------- max pool */
/* kxk window, stride s, no padding, floor mode.  First maximum in row-major
 * (ky then kx) scan wins (strict >); argmax stored as ky*k + kx. */
void orc_pool_fwd(const double* x, double* y, uint8_t* arg, int N, int C, int H, int W, int k, int s) {
    int Ho = (H - k) / s + 1, Wo = (W - k) / s + 1;
    #pragma omp parallel for
    for (int nc = 0; nc < N * C; ++nc) {
        const double* xp = x + (size_t)nc * H * W;
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox) {
                double best = xp[(oy * s) * W + ox * s];
                int bi = 0;
                for (int ky = 0; ky < k; ++ky)
                    for (int kx = 0; kx < k; ++kx) {
                        double v = xp[(oy * s + ky) * W + ox * s + kx];
                        if (v > best) { best = v; bi = ky * k + kx; }
                    }
                y[(size_t)nc * Ho * Wo + oy * Wo + ox] = best;
                arg[(size_t)nc * Ho * Wo + oy * Wo + ox] = (uint8_t)bi;
            }
    }
}

/* each dy is added at the argmax position of its window */
void orc_pool_bwd(const double* dy, const uint8_t* arg, double* dx, int N, int C, int H, int W, int k, int s) {
    int Ho = (H - k) / s + 1, Wo = (W - k) / s + 1;
    #pragma omp parallel for
    for (int nc = 0; nc < N * C; ++nc) {
        double* dxp = dx + (size_t)nc * H * W;
        for (int i = 0; i < H * W; ++i) dxp[i] = 0.0;
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox) {
                int a = arg[(size_t)nc * Ho * Wo + oy * Wo + ox];
                dxp[(oy * s + a / k) * W + ox * s + a % k] += dy[(size_t)nc * Ho * Wo + oy * Wo + ox];
            }
    }
}
