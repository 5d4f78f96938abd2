/*
 * CPU oracle for the CNN operator set of the Xenos paper (Table 3: x.conv, x.matmul,
 * x.gampool, x.add, x.concat, and the Conv-Bn-Relu members of x.cbr).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of every operator, run one
 * operator at a time on NCHW fp32 tensors with naive loops and fp32 accumulation.  It shares
 * no code, header, table or helper with the CUDA library and is never on the product path;
 * only the tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * The paper's optimiser emits "an optimized model equivalent to the original model"
 * (Section 3), and Eq. 1 is an identity, so the thing to check a linked / split execution
 * against is the unlinked definition written out below.
 *
 * Parallelism: OpenMP over the outermost (image x output-channel) loops only; the order in
 * which one output element sums its terms never depends on the thread count.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define XO_API __attribute__((visibility("default")))

XO_API int xo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

XO_API void xo_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Output extent of a strided window op: floor((in + 2*pad - k) / stride) + 1. */
XO_API int xo_out_dim(int in, int k, int stride, int pad) {
    int num = in + 2 * pad - k;
    if (num < 0) return 0;
    return num / stride + 1;
}

/*
 * x.conv (Table 3; Section 4.2.2 names the parameter dims K, C, R, S; Section 5 the seven
 * loop dims batch, inC, inH, inW, outC, r, s).
 *   y[n][k][p][q] = b[k] + sum_{c < C/g} sum_{r < R} sum_{s < S}
 *                   x[n][(k / (K/g)) * (C/g) + c][p*st - pad + r][q*st - pad + s] * w[k][c][r][s]
 * Taps that fall outside the input contribute nothing.  Depthwise is g = C = K.
 * Loop order n, k, p, q, c, r, s; one fp32 accumulator per output element, started at 0 and
 * the bias added last.
 */
XO_API void xo_conv2d(const float *x, int N, int C, int H, int W,
                      const float *w, int K, int R, int S,
                      int stride, int pad, int groups,
                      const float *bias, float *y) {
    const int P = xo_out_dim(H, R, stride, pad);
    const int Q = xo_out_dim(W, S, stride, pad);
    const int Cg = C / groups;
    const int Kg = K / groups;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int k = 0; k < K; ++k) {
            const int g = k / Kg;
            for (int p = 0; p < P; ++p) {
                for (int q = 0; q < Q; ++q) {
                    float acc = 0.0f;
                    for (int c = 0; c < Cg; ++c) {
                        const float *xc = x + ((size_t)n * C + (size_t)g * Cg + c) * H * W;
                        const float *wc = w + ((size_t)k * Cg + c) * R * S;
                        for (int r = 0; r < R; ++r) {
                            const int ih = p * stride - pad + r;
                            if (ih < 0 || ih >= H) continue;
                            for (int s = 0; s < S; ++s) {
                                const int iw = q * stride - pad + s;
                                if (iw < 0 || iw >= W) continue;
                                acc += xc[(size_t)ih * W + iw] * wc[r * S + s];
                            }
                        }
                    }
                    if (bias) acc += bias[k];
                    y[(((size_t)n * K + k) * P + p) * Q + q] = acc;
                }
            }
        }
    }
}

/*
 * Inference BatchNorm, the "Bn" of the paper's CBR operator (Section 4.3), kept un-folded:
 *   y = gamma * (x - mean) / sqrt(var + eps) + beta, per channel.
 */
XO_API void xo_batchnorm(const float *x, int N, int C, int HW,
                         const float *gamma, const float *beta,
                         const float *mean, const float *var, float eps, float *y) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < C; ++c) {
            const float inv = 1.0f / sqrtf(var[c] + eps);
            const float *xi = x + ((size_t)n * C + c) * HW;
            float *yi = y + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) yi[i] = gamma[c] * ((xi[i] - mean[c]) * inv) + beta[c];
        }
    }
}

/* The "Relu" of CBR: max(x, 0); and the clipped form min(max(x, 0), 6). */
XO_API void xo_relu(const float *x, size_t n, float *y) {
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) y[i] = x[i] > 0.0f ? x[i] : 0.0f;
}

XO_API void xo_relu6(const float *x, size_t n, float *y) {
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) {
        float v = x[i] > 0.0f ? x[i] : 0.0f;
        y[i] = v < 6.0f ? v : 6.0f;
    }
}

/* x.gampool, max form: maximum over the in-range elements of each window. */
XO_API void xo_maxpool(const float *x, int N, int C, int H, int W,
                       int k, int stride, int pad, float *y) {
    const int P = xo_out_dim(H, k, stride, pad);
    const int Q = xo_out_dim(W, k, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < C; ++c) {
            const float *xc = x + ((size_t)n * C + c) * H * W;
            float *yc = y + ((size_t)n * C + c) * P * Q;
            for (int p = 0; p < P; ++p) {
                for (int q = 0; q < Q; ++q) {
                    float m = -INFINITY;
                    for (int r = 0; r < k; ++r) {
                        const int ih = p * stride - pad + r;
                        if (ih < 0 || ih >= H) continue;
                        for (int s = 0; s < k; ++s) {
                            const int iw = q * stride - pad + s;
                            if (iw < 0 || iw >= W) continue;
                            const float v = xc[(size_t)ih * W + iw];
                            if (v > m) m = v;
                        }
                    }
                    yc[(size_t)p * Q + q] = m;
                }
            }
        }
    }
}

/* x.gampool, average form: mean over the in-range elements of each window. */
XO_API void xo_avgpool(const float *x, int N, int C, int H, int W,
                       int k, int stride, int pad, float *y) {
    const int P = xo_out_dim(H, k, stride, pad);
    const int Q = xo_out_dim(W, k, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < C; ++c) {
            const float *xc = x + ((size_t)n * C + c) * H * W;
            float *yc = y + ((size_t)n * C + c) * P * Q;
            for (int p = 0; p < P; ++p) {
                for (int q = 0; q < Q; ++q) {
                    float acc = 0.0f;
                    int cnt = 0;
                    for (int r = 0; r < k; ++r) {
                        const int ih = p * stride - pad + r;
                        if (ih < 0 || ih >= H) continue;
                        for (int s = 0; s < k; ++s) {
                            const int iw = q * stride - pad + s;
                            if (iw < 0 || iw >= W) continue;
                            acc += xc[(size_t)ih * W + iw];
                            ++cnt;
                        }
                    }
                    yc[(size_t)p * Q + q] = cnt ? acc / (float)cnt : 0.0f;
                }
            }
        }
    }
}

/* x.gampool, global form: mean over all H*W positions, sequential fp32 sum. y is [N][C]. */
XO_API void xo_global_avgpool(const float *x, int N, int C, int HW, float *y) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < C; ++c) {
            const float *xi = x + ((size_t)n * C + c) * HW;
            float acc = 0.0f;
            for (int i = 0; i < HW; ++i) acc += xi[i];
            y[(size_t)n * C + c] = acc / (float)HW;
        }
    }
}

/* x.add: element-wise a + b. */
XO_API void xo_add(const float *a, const float *b, size_t n, float *y) {
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) y[i] = a[i] + b[i];
}

/*
 * x.concat along channels: writes one input of Ci channels at channel offset coff of an
 * output with Ctot channels.  Calling it once per input, in argument order, is the concat.
 */
XO_API void xo_concat_part(const float *x, int N, int Ci, int HW, int Ctot, int coff, float *y) {
    for (int n = 0; n < N; ++n)
        memcpy(y + ((size_t)n * Ctot + coff) * HW, x + (size_t)n * Ci * HW,
               (size_t)Ci * HW * sizeof(float));
}

/* x.matmul as the fully connected layer of Eq. 1: y = W x + B, W is [K][C], x is [N][C]. */
XO_API void xo_fc(const float *x, int N, int C, const float *w, int K, const float *bias, float *y) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int k = 0; k < K; ++k) {
            float acc = 0.0f;
            for (int c = 0; c < C; ++c) acc += w[(size_t)k * C + c] * x[(size_t)n * C + c];
            if (bias) acc += bias[k];
            y[(size_t)n * K + k] = acc;
        }
    }
}

/* x.mul (Table 3): element-wise a * b. */
XO_API void xo_mul(const float *a, const float *b, size_t n, float *y) {
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) y[i] = a[i] * b[i];
}

/* x.mac (Table 3): element-wise multiply accumulate, a * b + c; the product is a rounded fp32 value. */
XO_API void xo_mac(const float *a, const float *b, const float *c, size_t n, float *y) {
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) {
        float p = a[i] * b[i];
        y[i] = p + c[i];
    }
}

/*
 * x.transpose (Table 3) of one matrix per image.  A matrix is a feature map of width 1, rows = H, columns = C,
 * stored NCHW as x[n][c][h]; the result has rows = C, columns = H: y[n][h][c] = x[n][c][h].
 */
XO_API void xo_transpose(const float *x, int N, int C, int H, float *y) {
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h) y[((size_t)n * H + h) * C + c] = x[((size_t)n * C + c) * H + h];
}

/* x.split (Table 3), one part: channels [coff, coff + Ci) of an input with Ctot channels. */
XO_API void xo_split_part(const float *x, int N, int Ci, int HW, int Ctot, int coff, float *y) {
    for (int n = 0; n < N; ++n)
        memcpy(y + (size_t)n * Ci * HW, x + ((size_t)n * Ctot + coff) * HW, (size_t)Ci * HW * sizeof(float));
}

/*
 * x.matmul (Table 3): A * B (+ bias) per image.  A has R rows of K columns and is stored as the feature map
 * a[n][k][r] (channels = columns); B is the constant [K][M] matrix, row-major; y[n][m][r] = sum_k a[n][k][r] * B[k][m].
 */
XO_API void xo_matmul(const float *a, int N, int K, int R, const float *b, int M, const float *bias, float *y) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            for (int r = 0; r < R; ++r) {
                float acc = 0.0f;
                for (int k = 0; k < K; ++k) acc += a[((size_t)n * K + k) * R + r] * b[(size_t)k * M + m];
                if (bias) acc += bias[m];
                y[((size_t)n * M + m) * R + r] = acc;
            }
        }
    }
}

/*
 * Diagnostic only: round an fp32 array to the nearest bf16 value (ties to even), kept in
 * fp32.  Lets a test separate precision drift of a bf16 execution from an indexing bug.
 */
XO_API void xo_round_bf16(const float *x, size_t n, float *y) {
    for (size_t i = 0; i < n; ++i) {
        uint32_t u;
        memcpy(&u, &x[i], 4);
        if ((u & 0x7f800000u) != 0x7f800000u) {
            uint32_t lsb = (u >> 16) & 1u;
            u += 0x7fffu + lsb;
        }
        u &= 0xffff0000u;
        memcpy(&y[i], &u, 4);
    }
}

/* ------------------------------------------------------------------------------------------
 * Linked (tile-by-tile) evaluation of a chain, restated in plain loops.
 *
 * Section 4.1: the producer hands its consumer exactly the elements the consumer reads, in
 * the consumer's order; for a k x k consumer the hand-over "replicates" the elements shared
 * by neighbouring windows.  Evaluated tile by tile, that is: to produce an output tile of the
 * last stage, take the window of stage i-1 outputs it reads (the halo), recursively, and
 * evaluate every stage on just that window.  Elements in the overlap of two tiles' windows
 * are evaluated once per tile.  Every element is summed in the same order as in xo_conv2d,
 * so the result must equal the one-operator-at-a-time result exactly.
 *
 * A stage is  conv(+bias) [-> batchnorm] [-> relu | relu6]   or   max/avg pool.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t kind;    /* 0 conv, 1 max pool, 2 avg pool */
    int32_t cout;    /* conv: K; pool: ignored (channels pass through) */
    int32_t k, stride, pad, groups;
    int32_t act;     /* 0 none, 1 relu, 2 relu6 */
    int32_t has_bn;
    const float *w, *bias, *gamma, *beta, *mean, *var;
    float eps;
} xo_stage_t;

typedef struct { int lo_h, hi_h, lo_w, hi_w; } xo_win_t;   /* half-open, may leave [0, dim) */

/* Window of stage-input coordinates read by the output window `o` of one stage. */
static xo_win_t xo_need(const xo_stage_t *s, xo_win_t o) {
    xo_win_t i;
    i.lo_h = o.lo_h * s->stride - s->pad;
    i.hi_h = (o.hi_h - 1) * s->stride - s->pad + s->k;
    i.lo_w = o.lo_w * s->stride - s->pad;
    i.hi_w = (o.hi_w - 1) * s->stride - s->pad + s->k;
    return i;
}

static int xo_clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

/*
 * Evaluate one stage for image n on an output window.  `in` holds the stage input on window
 * `iw_` (clipped to the real extent Hin x Win), channel-major [C][ih][iw]; out-of-range
 * positions are simply absent and are treated exactly as the definitions above treat them.
 */
static void xo_stage_eval(const xo_stage_t *s, const float *in, int C, int Hin, int Win,
                          xo_win_t iwin, xo_win_t owin, float *out, int *Cout) {
    const int ih0 = iwin.lo_h, iw0 = iwin.lo_w;
    const int IH = iwin.hi_h - iwin.lo_h, IW = iwin.hi_w - iwin.lo_w;
    const int OH = owin.hi_h - owin.lo_h, OW = owin.hi_w - owin.lo_w;
    if (s->kind == 0) {
        const int K = s->cout, Cg = C / s->groups, Kg = K / s->groups;
        *Cout = K;
        for (int k = 0; k < K; ++k) {
            const int g = k / Kg;
            float inv = 0.0f;
            if (s->has_bn) inv = 1.0f / sqrtf(s->var[k] + s->eps);
            for (int p = owin.lo_h; p < owin.hi_h; ++p) {
                for (int q = owin.lo_w; q < owin.hi_w; ++q) {
                    float acc = 0.0f;
                    for (int c = 0; c < Cg; ++c) {
                        const float *xc = in + (size_t)(g * Cg + c) * IH * IW;
                        const float *wc = s->w + ((size_t)k * Cg + c) * s->k * s->k;
                        for (int r = 0; r < s->k; ++r) {
                            const int ih = p * s->stride - s->pad + r;
                            if (ih < 0 || ih >= Hin) continue;
                            for (int t = 0; t < s->k; ++t) {
                                const int iw = q * s->stride - s->pad + t;
                                if (iw < 0 || iw >= Win) continue;
                                acc += xc[(size_t)(ih - ih0) * IW + (iw - iw0)] * wc[r * s->k + t];
                            }
                        }
                    }
                    if (s->bias) acc += s->bias[k];
                    if (s->has_bn) acc = s->gamma[k] * ((acc - s->mean[k]) * inv) + s->beta[k];
                    if (s->act >= 1) acc = acc > 0.0f ? acc : 0.0f;
                    if (s->act == 2) acc = acc < 6.0f ? acc : 6.0f;
                    out[((size_t)k * OH + (p - owin.lo_h)) * OW + (q - owin.lo_w)] = acc;
                }
            }
        }
    } else {
        *Cout = C;
        for (int c = 0; c < C; ++c) {
            const float *xc = in + (size_t)c * IH * IW;
            for (int p = owin.lo_h; p < owin.hi_h; ++p) {
                for (int q = owin.lo_w; q < owin.hi_w; ++q) {
                    float m = -INFINITY, acc = 0.0f;
                    int cnt = 0;
                    for (int r = 0; r < s->k; ++r) {
                        const int ih = p * s->stride - s->pad + r;
                        if (ih < 0 || ih >= Hin) continue;
                        for (int t = 0; t < s->k; ++t) {
                            const int iw = q * s->stride - s->pad + t;
                            if (iw < 0 || iw >= Win) continue;
                            const float v = xc[(size_t)(ih - ih0) * IW + (iw - iw0)];
                            if (v > m) m = v;
                            acc += v;
                            ++cnt;
                        }
                    }
                    out[((size_t)c * OH + (p - owin.lo_h)) * OW + (q - owin.lo_w)] =
                        s->kind == 1 ? m : (cnt ? acc / (float)cnt : 0.0f);
                }
            }
        }
    }
}

/*
 * Run `ns` stages on x[N][C][H][W] with the LAST stage's output cut into tiles of th x tw.
 * Writes y (NCHW of the last stage).  If halo_out is non-NULL it receives, for the first tile
 * of image 0, the clipped input window of every stage: 4 ints per stage (lo_h, hi_h, lo_w,
 * hi_w) so a test can compare it with a brute-force receptive field.
 * Returns 0, or -1 on allocation failure / bad arguments.
 */
XO_API int xo_chain_tiled(const float *x, int N, int C, int H, int W,
                          const xo_stage_t *st, int ns, int th, int tw,
                          float *y, int32_t *halo_out) {
    if (ns < 1 || ns > 8 || th < 1 || tw < 1) return -1;
    int ch[9], hh[9], ww[9];
    ch[0] = C; hh[0] = H; ww[0] = W;
    for (int i = 0; i < ns; ++i) {
        ch[i + 1] = st[i].kind == 0 ? st[i].cout : ch[i];
        hh[i + 1] = xo_out_dim(hh[i], st[i].k, st[i].stride, st[i].pad);
        ww[i + 1] = xo_out_dim(ww[i], st[i].k, st[i].stride, st[i].pad);
    }
    const int OH = hh[ns], OW = ww[ns], OC = ch[ns];
    int rc = 0;
    for (int n = 0; n < N && rc == 0; ++n) {
        for (int t0 = 0; t0 < OH && rc == 0; t0 += th) {
            for (int u0 = 0; u0 < OW && rc == 0; u0 += tw) {
                /* windows, from the last stage's output tile back to the chain input */
                xo_win_t win[9];
                win[ns].lo_h = t0; win[ns].hi_h = t0 + th < OH ? t0 + th : OH;
                win[ns].lo_w = u0; win[ns].hi_w = u0 + tw < OW ? u0 + tw : OW;
                for (int i = ns - 1; i >= 0; --i) {
                    xo_win_t need = xo_need(&st[i], win[i + 1]);
                    win[i].lo_h = xo_clampi(need.lo_h, 0, hh[i]);
                    win[i].hi_h = xo_clampi(need.hi_h, 0, hh[i]);
                    win[i].lo_w = xo_clampi(need.lo_w, 0, ww[i]);
                    win[i].hi_w = xo_clampi(need.hi_w, 0, ww[i]);
                }
                if (halo_out && n == 0 && t0 == 0 && u0 == 0) {
                    for (int i = 0; i < ns; ++i) {
                        halo_out[4 * i + 0] = win[i].lo_h; halo_out[4 * i + 1] = win[i].hi_h;
                        halo_out[4 * i + 2] = win[i].lo_w; halo_out[4 * i + 3] = win[i].hi_w;
                    }
                }
                /* copy the chain-input window of image n */
                int IH = win[0].hi_h - win[0].lo_h, IW = win[0].hi_w - win[0].lo_w;
                float *cur = (float *)malloc(sizeof(float) * (size_t)ch[0] * IH * IW + 16);
                if (!cur) { rc = -1; break; }
                for (int c = 0; c < ch[0]; ++c)
                    for (int i = 0; i < IH; ++i)
                        memcpy(cur + ((size_t)c * IH + i) * IW,
                               x + (((size_t)n * C + c) * H + win[0].lo_h + i) * W + win[0].lo_w,
                               sizeof(float) * (size_t)IW);
                for (int i = 0; i < ns; ++i) {
                    const int oh = win[i + 1].hi_h - win[i + 1].lo_h;
                    const int ow = win[i + 1].hi_w - win[i + 1].lo_w;
                    float *nxt = (float *)malloc(sizeof(float) * (size_t)ch[i + 1] * oh * ow + 16);
                    if (!nxt) { rc = -1; break; }
                    int co = 0;
                    xo_stage_eval(&st[i], cur, ch[i], hh[i], ww[i], win[i], win[i + 1], nxt, &co);
                    free(cur);
                    cur = nxt;
                }
                if (rc == 0) {
                    const int oh = win[ns].hi_h - win[ns].lo_h, ow = win[ns].hi_w - win[ns].lo_w;
                    for (int c = 0; c < OC; ++c)
                        for (int i = 0; i < oh; ++i)
                            memcpy(y + (((size_t)n * OC + c) * OH + win[ns].lo_h + i) * OW + win[ns].lo_w,
                                   cur + ((size_t)c * oh + i) * ow, sizeof(float) * (size_t)ow);
                }
                free(cur);
            }
        }
    }
    return rc;
}

XO_API size_t xo_stage_struct_size(void) { return sizeof(xo_stage_t); }
