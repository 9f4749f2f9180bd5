/*
 * CPU oracle for the cached causal Conv3D forward pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition against
 * which the CUDA library is checked.  It shares no code with the CUDA path and
 * must never be linked into, imported by or called from the product.
 *
 * What it computes (the paper's Section 4.1/4.2, Eq. (1) "source time" and
 * Eq. (2) "conv3d", with the effective left pad p_l = p_l^base - |C|_T = 0 for
 * a cache that holds kt-1 frames):
 *
 *   Z[n,ci,tau,h,w]  = cache[n,ci,tau,h,w]             0 <= tau < kt-1   (zeros if cache == NULL)
 *                    = x[n,ci,tau-(kt-1),h,w]          kt-1 <= tau < kt-1+T
 *   out[n,co,t,h,w]  = b[co] + sum_{ci,dt,dh,dw} w[co,ci,dt,dh,dw] * Z[n,ci,t+dt,h+dh-ph,w+dw-pw]
 *                      (cross-correlation; terms whose spatial source is outside [0,H)x[0,W) are zero;
 *                       ph=(kh-1)/2, pw=(kw-1)/2; bias added exactly once)
 *   new_cache[n,ci,j,h,w] = Z[n,ci,T+j,h,w]            0 <= j < kt-1
 *
 * Arithmetic: every stored input (fp32, or bf16 given as its 16-bit pattern)
 * is widened exactly to double; every product and sum is a double; per output
 * element the order is bias first, then (ci,dt,dh,dw) lexicographic, whatever
 * the thread count.  The output is returned in double and is never rounded.
 * The cache update is a bit copy.
 *
 * Parity pins (tests/test_oracle_*.py): hand-computed examples under
 * tests/golden/, a structurally different brute-force routine, Eq. (2) read
 * frame by frame (one library 2-D correlation per output frame and temporal
 * tap at the source time of Eq. (1)), the fp64 library conv3d on the explicitly
 * concatenated input, and the invariants (causality, streaming equivalence,
 * linearity, 1x1x1 = per-pixel matmul, delta kernel).
 * Parity unpinned: behaviour on NaN/Inf/subnormal inputs.
 *
 * ccv3d_oracle_forward_general (end of file) is the same operator with the
 * layer's own spatial stride, padding and dilation and a temporal dilation
 * (Eq. (1)-(2) as printed); its pins are in tests/test_oracle_general.py:
 * hand-worked values, bit-for-bit reduction to ccv3d_oracle_forward, a numpy
 * routine of different structure, the fp64 library conv3d, Eq. (4)'s interval
 * route, streaming equivalence and causality under temporal dilation.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_BF16 = 1 };

static inline double widen(const void* p, int dtype, int64_t i) {
    if (dtype == ORC_BF16) {
        uint32_t u = ((uint32_t)((const uint16_t*)p)[i]) << 16;
        float f;
        memcpy(&f, &u, 4);
        return (double)f;
    }
    return (double)((const float*)p)[i];
}

static inline size_t esize(int dtype) { return dtype == ORC_BF16 ? 2 : 4; }

/* Frame tau of Z = [cache ; x] for sample n, channel ci: pointer to H*W stored
 * elements, or NULL when the frame is an absent (zero) cache frame. */
static inline const char* z_frame(const void* x, const void* cache, int dtype, int Cin, int T, int64_t HW,
                                  int kt, int n, int ci, int tau) {
    const int tc = kt - 1;
    if (tau < tc) {
        if (!cache) return NULL;
        return (const char*)cache + (size_t)((((int64_t)n * Cin + ci) * tc + tau) * HW) * esize(dtype);
    }
    return (const char*)x + (size_t)((((int64_t)n * Cin + ci) * T + (tau - tc)) * HW) * esize(dtype);
}

/* Full forward.  out: double[N,Cout,T,H,W].  new_cache (may be NULL): same
 * dtype as x, [N,Cin,kt-1,H,W].  b may be NULL (zero bias).  Returns 0, or -1
 * on bad arguments. */
int ccv3d_oracle_forward(int dtype, const void* x, const void* cache, const void* w, const void* b,
                         int N, int Cin, int Cout, int T, int H, int W, int kt, int kh, int kw,
                         double* out, void* new_cache) {
    if (!x || !w || !out || N < 1 || Cin < 1 || Cout < 1 || T < 1 || H < 1 || W < 1) return -1;
    if (kt < 1 || kh < 1 || kw < 1 || !(kh & 1) || !(kw & 1)) return -1;
    const int ph = (kh - 1) / 2, pw = (kw - 1) / 2;
    const int64_t HW = (int64_t)H * W;
    const int64_t work = (int64_t)N * Cout * T;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t it = 0; it < work; ++it) {
        const int t = (int)(it % T);
        const int co = (int)((it / T) % Cout);
        const int n = (int)(it / ((int64_t)T * Cout));
        double* acc = out + it * HW; /* (n,co,t) plane, already in NCTHW order */
        const double bias = b ? widen(b, dtype, co) : 0.0;
        for (int64_t i = 0; i < HW; ++i) acc[i] = bias;
        for (int ci = 0; ci < Cin; ++ci)
            for (int dt = 0; dt < kt; ++dt) {
                const char* zf = z_frame(x, cache, dtype, Cin, T, HW, kt, n, ci, t + dt);
                if (!zf) continue; /* absent cache frame: every term is an exact zero */
                for (int dh = 0; dh < kh; ++dh)
                    for (int dw = 0; dw < kw; ++dw) {
                        const double wv =
                            widen(w, dtype, ((((int64_t)co * Cin + ci) * kt + dt) * kh + dh) * kw + dw);
                        const int h_lo = ph - dh > 0 ? ph - dh : 0;
                        const int h_hi = H + ph - dh < H ? H + ph - dh : H;
                        const int w_lo = pw - dw > 0 ? pw - dw : 0;
                        const int w_hi = W + pw - dw < W ? W + pw - dw : W;
                        for (int h = h_lo; h < h_hi; ++h) {
                            double* arow = acc + (int64_t)h * W;
                            const int64_t src = (int64_t)(h + dh - ph) * W + (dw - pw);
                            if (dtype == ORC_BF16) {
                                const uint16_t* zr = (const uint16_t*)zf + src;
                                for (int ww = w_lo; ww < w_hi; ++ww) {
                                    uint32_t u = ((uint32_t)zr[ww]) << 16;
                                    float f;
                                    memcpy(&f, &u, 4);
                                    arow[ww] += wv * (double)f;
                                }
                            } else {
                                const float* zr = (const float*)zf + src;
                                for (int ww = w_lo; ww < w_hi; ++ww) arow[ww] += wv * (double)zr[ww];
                            }
                        }
                    }
            }
    }

    if (new_cache && kt > 1) {
        const int tc = kt - 1;
        const size_t fb = (size_t)HW * esize(dtype);
        for (int n = 0; n < N; ++n)
            for (int ci = 0; ci < Cin; ++ci)
                for (int j = 0; j < tc; ++j) {
                    char* dst = (char*)new_cache + (size_t)(((int64_t)n * Cin + ci) * tc + j) * fb;
                    const char* zf = z_frame(x, cache, dtype, Cin, T, HW, kt, n, ci, T + j);
                    if (zf) memcpy(dst, zf, fb);
                    else memset(dst, 0, fb);
                }
    }
    return 0;
}

/* The same definition evaluated one output element at a time, for sampled
 * checks of problems too large to run whole.  idx[i] is a flat index into
 * out[N,Cout,T,H,W]; vals[i] receives that element. */
int ccv3d_oracle_points(int dtype, const void* x, const void* cache, const void* w, const void* b,
                        int N, int Cin, int Cout, int T, int H, int W, int kt, int kh, int kw,
                        const int64_t* idx, int64_t npts, double* vals) {
    if (!x || !w || !idx || !vals) return -1;
    const int ph = (kh - 1) / 2, pw = (kw - 1) / 2;
    const int64_t HW = (int64_t)H * W;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t p = 0; p < npts; ++p) {
        int64_t r = idx[p];
        const int ww = (int)(r % W); r /= W;
        const int h = (int)(r % H); r /= H;
        const int t = (int)(r % T); r /= T;
        const int co = (int)(r % Cout); r /= Cout;
        const int n = (int)r;
        double acc = b ? widen(b, dtype, co) : 0.0;
        for (int ci = 0; ci < Cin; ++ci)
            for (int dt = 0; dt < kt; ++dt) {
                const char* zf = z_frame(x, cache, dtype, Cin, T, HW, kt, n, ci, t + dt);
                if (!zf) continue;
                for (int dh = 0; dh < kh; ++dh) {
                    const int hs = h + dh - ph;
                    if (hs < 0 || hs >= H) continue;
                    for (int dw = 0; dw < kw; ++dw) {
                        const int ws = ww + dw - pw;
                        if (ws < 0 || ws >= W) continue;
                        const double wv =
                            widen(w, dtype, ((((int64_t)co * Cin + ci) * kt + dt) * kh + dh) * kw + dw);
                        acc += wv * widen(zf, dtype, (int64_t)hs * W + ws);
                    }
                }
            }
        vals[p] = acc;
    }
    return 0;
}

/* The cache update alone (the last kt-1 frames of Z = [cache ; x], bit copy), for problems whose full
 * forward pass is too large to run on the CPU. */
int ccv3d_oracle_cache_update(int dtype, const void* x, const void* cache, int N, int Cin, int T, int H, int W, int kt,
                              void* new_cache) {
    if (!x || !new_cache || kt < 2) return -1;
    const int tc = kt - 1;
    const int64_t HW = (int64_t)H * W;
    const size_t fb = (size_t)HW * esize(dtype);
    for (int n = 0; n < N; ++n)
        for (int ci = 0; ci < Cin; ++ci)
            for (int j = 0; j < tc; ++j) {
                char* dst = (char*)new_cache + (size_t)(((int64_t)n * Cin + ci) * tc + j) * fb;
                const char* zf = z_frame(x, cache, dtype, Cin, T, HW, kt, n, ci, T + j);
                if (zf) memcpy(dst, zf, fb);
                else memset(dst, 0, fb);
            }
    return 0;
}

int ccv3d_oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------------
 * The operator with the paper's full supported contract (Section 4.1, Eq. (1)-(2) as printed): original
 * spatial stride s = (s_h, s_w), padding p = (p_h, p_w) and dilation d = (d_h, d_w) inside every temporal
 * tap's 2-D correlation, temporal dilation d_t in the source time q_k(t) = t + k d_t - p_l, unit temporal
 * stride, one group.  The causal pad is p_l^base = d_t (kt-1) frames; the cache holds the newest cf of them
 * (0 <= cf <= d_t (kt-1)), older ones do not exist and contribute zero:
 *
 *   tc = d_t (kt-1)
 *   Z[n,ci,tau]      = 0                          0 <= tau < tc-cf
 *                    = cache[n,ci,tau-(tc-cf)]    tc-cf <= tau < tc
 *                    = x[n,ci,tau-tc]             tc <= tau < tc+T
 *   H_o = floor((H + 2 p_h - d_h (kh-1) - 1) / s_h) + 1,   W_o likewise
 *   out[n,co,t,ho,wo] = b[co] + sum_{ci,k,dh,dw} w[co,ci,k,dh,dw]
 *                                * Z[n,ci, t + k d_t, ho s_h + dh d_h - p_h, wo s_w + dw d_w - p_w]
 *   new_cache[n,ci,j] = Z[n,ci,T+j]               0 <= j < tc
 *
 * Written separately from ccv3d_oracle_forward (which it must reproduce bit for bit at s = d = d_t = 1,
 * p = (k-1)/2, cf = kt-1: a test holds it to that), output-element-outermost, same arithmetic rules: exact
 * widening, double products and sums, bias first, then (ci, k, dh, dw) lexicographic.
 * ------------------------------------------------------------------------------------------------ */
typedef struct {
    int N, Cin, Cout, T, H, W;
    int kt, kh, kw;
    int sh, sw, ph, pw, dh, dw, dil_t;
    int cf; /* frames the cache holds */
    int st; /* temporal stride (the paper's method itself handles 1 only; Eq. (3) "output time" is printed for any s_t) */
} orc_geom;

static inline int out_extent(int in, int pad, int dil, int k, int stride) {
    const int span = in + 2 * pad - dil * (k - 1) - 1;
    return span < 0 ? 0 : span / stride + 1;
}

static inline const char* zg_frame(const orc_geom* g, int dtype, const void* x, const void* cache, int n, int ci,
                                   int tau) {
    const int tc = g->dil_t * (g->kt - 1);
    const int64_t HW = (int64_t)g->H * g->W;
    if (tau < tc) {
        const int cfr = tau - (tc - g->cf);
        if (!cache || cfr < 0) return NULL;
        return (const char*)cache + (size_t)((((int64_t)n * g->Cin + ci) * g->cf + cfr) * HW) * esize(dtype);
    }
    return (const char*)x + (size_t)((((int64_t)n * g->Cin + ci) * g->T + (tau - tc)) * HW) * esize(dtype);
}

static int geom_ok(const orc_geom* g) {
    if (g->N < 1 || g->Cin < 1 || g->Cout < 1 || g->T < 1 || g->H < 1 || g->W < 1) return 0;
    if (g->kt < 1 || g->kh < 1 || g->kw < 1) return 0;
    if (g->sh < 1 || g->sw < 1 || g->dh < 1 || g->dw < 1 || g->dil_t < 1 || g->ph < 0 || g->pw < 0 || g->st < 1) return 0;
    if (g->cf < 0 || g->cf > g->dil_t * (g->kt - 1)) return 0;
    return 1;
}

/* T_o of the output-time equation with |Z| + p_l = d_t (kt-1) + T and p_r = 0: floor((T - 1) / s_t) + 1. */
static inline int out_frames(const orc_geom* g) { return (g->T - 1) / g->st + 1; }

int ccv3d_oracle_out_dims(const orc_geom* g, int* To, int* Ho, int* Wo) {
    if (!g || !geom_ok(g)) return -1;
    *To = out_frames(g);
    *Ho = out_extent(g->H, g->ph, g->dh, g->kh, g->sh);
    *Wo = out_extent(g->W, g->pw, g->dw, g->kw, g->sw);
    return 0;
}

/* With a temporal stride s_t the source time of tap k for output frame o is o s_t + k d_t (in Z), and there are T_o
 * output frames.  out: double[N,Cout,T_o,H_o,W_o]; new_cache (may be NULL): [N,Cin,d_t(kt-1),H,W] in the storage dtype. */
int ccv3d_oracle_forward_general(int dtype, const void* x, const void* cache, const void* w, const void* b,
                                 const orc_geom* g, double* out, void* new_cache) {
    if (!x || !w || !out || !g || !geom_ok(g)) return -1;
    if (g->cf > 0 && !cache) return -1;
    const int Ho = out_extent(g->H, g->ph, g->dh, g->kh, g->sh), Wo = out_extent(g->W, g->pw, g->dw, g->kw, g->sw);
    const int tc = g->dil_t * (g->kt - 1);
    const int To = out_frames(g);
    const int64_t total = (int64_t)g->N * g->Cout * To * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < total; ++e) {
        int64_t r = e;
        const int wo = (int)(r % Wo); r /= Wo;
        const int ho = (int)(r % Ho); r /= Ho;
        const int t = (int)(r % To); r /= To;
        const int co = (int)(r % g->Cout);
        const int n = (int)(r / g->Cout);
        double acc = b ? widen(b, dtype, co) : 0.0;
        for (int ci = 0; ci < g->Cin; ++ci)
            for (int k = 0; k < g->kt; ++k) {
                const char* zf = zg_frame(g, dtype, x, cache, n, ci, t * g->st + k * g->dil_t);
                if (!zf) continue;
                for (int a = 0; a < g->kh; ++a) {
                    const int hs = ho * g->sh + a * g->dh - g->ph;
                    if (hs < 0 || hs >= g->H) continue;
                    for (int c = 0; c < g->kw; ++c) {
                        const int ws = wo * g->sw + c * g->dw - g->pw;
                        if (ws < 0 || ws >= g->W) continue;
                        const double wv =
                            widen(w, dtype, ((((int64_t)co * g->Cin + ci) * g->kt + k) * g->kh + a) * g->kw + c);
                        acc += wv * widen(zf, dtype, (int64_t)hs * g->W + ws);
                    }
                }
            }
        out[e] = acc;
    }
    if (new_cache && tc > 0) {
        const size_t fb = (size_t)g->H * g->W * esize(dtype);
        for (int n = 0; n < g->N; ++n)
            for (int ci = 0; ci < g->Cin; ++ci)
                for (int j = 0; j < tc; ++j) {
                    char* dst = (char*)new_cache + (size_t)(((int64_t)n * g->Cin + ci) * tc + j) * fb;
                    const char* zf = zg_frame(g, dtype, x, cache, n, ci, g->T + j);
                    if (zf) memcpy(dst, zf, fb);
                    else memset(dst, 0, fb);
                }
    }
    return 0;
}
