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
 * tests/golden/, a structurally different brute-force routine, a literal
 * per-tap Algorithm-1 route, the fp64 library conv3d on the explicitly
 * concatenated input, and the invariants (causality, streaming equivalence,
 * linearity, 1x1x1 = per-pixel matmul, delta kernel).
 * Parity unpinned: behaviour on NaN/Inf/subnormal inputs.
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
