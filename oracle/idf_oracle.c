/*
 * Oracle: conventional layer-by-layer CNN inference (test infrastructure only).
 *
 * This file is the plain definition the incremental depth-first scheme must
 * reproduce: the paper states that the incremental output is identical to the
 * output of the conventional network (Introduction; Section "Asynchronous
 * incremental updates", the paragraph after Eq. 5), so the reference result is
 * Eq. 1 applied one whole layer at a time, h(n) = f(W h(n-1) + b), with the sum
 * over j restricted to the convolution kernel's neighbourhood (the paragraph
 * that introduces convolutions after Eq. 5).
 *
 * It is deliberately slow and obvious: no blocking, no fusion, no intrinsics.
 * Floating-point nets accumulate in double; integer nets in int32.
 * Nothing in the product path may call into this file.  Only tests, the smoke
 * check and the CPU-baseline timing leg of the benchmark do.
 *
 * Layouts (channels innermost everywhere):
 *   maps     [n_streams][H][W][C]
 *   weights  [Cout][Kh][Kw][Cin]      (cross-correlation, no kernel flip)
 * Zero padding of `pad` on all four sides, the same stride on both axes,
 * output size floor((H + 2 pad - Kh) / stride) + 1.  A 1D net is W = Kw = 1:
 * its x axis is degenerate and takes neither padding nor stride.
 *
 * Pins (tests that do not depend on this file's own arithmetic):
 *   - torch.nn.functional conv/relu/max_pool2d in float64 on CPU,
 *   - single-unit brute-force sums written separately in the tests,
 *   - impulse / all-ones closed forms, linearity, positive homogeneity,
 *   - the event-by-event implementation in idf_event_checker.c,
 *   - bf16 rounding against torch's float32->bfloat16 conversion,
 *   - requantisation against exact rational arithmetic in Python.
 */
#include <stdint.h>
#include <string.h>
#include <math.h>

/* Eq. 1 for one convolutional layer, floating point.
 * out[s][oy][ox][co] = f( b[co] + sum_{ky,kx,ci} w[co][ky][kx][ci] * in[s][oy*st-p+ky][ox*st-p+kx][ci] )
 * with in == 0 outside the map; f = ReLU when relu != 0, identity otherwise. */
void orc_conv_f64(const double* in, long long n_streams, int H, int W, int Cin,
                  const double* w, const double* b, int Cout, int Kh, int Kw,
                  int stride, int pad, int relu, double* out)
{
    const int one_d = (W == 1 && Kw == 1);
    const int pad_x = one_d ? 0 : pad, stride_x = one_d ? 1 : stride;
    const int Ho = (H + 2 * pad - Kh) / stride + 1;
    const int Wo = (W + 2 * pad_x - Kw) / stride_x + 1;
    if (H + 2 * pad < Kh || W + 2 * pad_x < Kw) return;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long s = 0; s < n_streams; ++s) {
        const double* ins = in + (size_t)s * H * W * Cin;
        double* outs = out + (size_t)s * Ho * Wo * Cout;
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox)
                for (int co = 0; co < Cout; ++co) {
                    double c = b ? b[co] : 0.0;
                    for (int ky = 0; ky < Kh; ++ky) {
                        const int iy = oy * stride - pad + ky;
                        if (iy < 0 || iy >= H) continue;
                        for (int kx = 0; kx < Kw; ++kx) {
                            const int ix = ox * stride_x - pad_x + kx;
                            if (ix < 0 || ix >= W) continue;
                            const double* a = ins + ((size_t)iy * W + ix) * Cin;
                            const double* ww = w + (((size_t)co * Kh + ky) * Kw + kx) * Cin;
                            for (int ci = 0; ci < Cin; ++ci) c += ww[ci] * a[ci];
                        }
                    }
                    if (relu && c < 0.0) c = 0.0;
                    outs[((size_t)oy * Wo + ox) * Cout + co] = c;
                }
    }
}

/* Eq. 1 for one convolutional layer, integer nets: int32 accumulator, values
 * of `in` and `w` lie in the int8 range so the sum cannot overflow for the
 * supported fan-ins.  Returns the raw state c (after ReLU if requested);
 * orc_requant_i32 turns it into the int8-range activation. */
void orc_conv_i32(const int32_t* in, long long n_streams, int H, int W, int Cin,
                  const int32_t* w, const int32_t* b, int Cout, int Kh, int Kw,
                  int stride, int pad, int relu, int32_t* out)
{
    const int one_d = (W == 1 && Kw == 1);
    const int pad_x = one_d ? 0 : pad, stride_x = one_d ? 1 : stride;
    const int Ho = (H + 2 * pad - Kh) / stride + 1;
    const int Wo = (W + 2 * pad_x - Kw) / stride_x + 1;
    if (H + 2 * pad < Kh || W + 2 * pad_x < Kw) return;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long s = 0; s < n_streams; ++s) {
        const int32_t* ins = in + (size_t)s * H * W * Cin;
        int32_t* outs = out + (size_t)s * Ho * Wo * Cout;
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox)
                for (int co = 0; co < Cout; ++co) {
                    int32_t c = b ? b[co] : 0;
                    for (int ky = 0; ky < Kh; ++ky) {
                        const int iy = oy * stride - pad + ky;
                        if (iy < 0 || iy >= H) continue;
                        for (int kx = 0; kx < Kw; ++kx) {
                            const int ix = ox * stride_x - pad_x + kx;
                            if (ix < 0 || ix >= W) continue;
                            const int32_t* a = ins + ((size_t)iy * W + ix) * Cin;
                            const int32_t* ww = w + (((size_t)co * Kh + ky) * Kw + kx) * Cin;
                            for (int ci = 0; ci < Cin; ++ci) c += ww[ci] * a[ci];
                        }
                    }
                    if (relu && c < 0) c = 0;
                    outs[((size_t)oy * Wo + ox) * Cout + co] = c;
                }
    }
}

/* Activation quantiser of the integer nets (the paper only mentions low
 * precision in passing and fixes no scheme; this one is ours):
 *   q = clamp( floor( (c + 2^(shift-1)) / 2^shift ), lo, 127 ),  lo = 0 after ReLU, -127 otherwise;
 * shift == 0 means no rounding term.  floor division == arithmetic shift. */
void orc_requant_i32(int32_t* c, long long n, int shift, int relu)
{
    const int32_t lo = relu ? 0 : -127;
    for (long long i = 0; i < n; ++i) {
        int64_t v = c[i];
        if (shift > 0) {
            v += (int64_t)1 << (shift - 1);
            /* floor division by 2^shift, written without relying on >> of negatives */
            int64_t d = (int64_t)1 << shift;
            int64_t q = v / d;
            if ((v % d) != 0 && v < 0) q -= 1;
            v = q;
        }
        if (v < lo) v = lo;
        if (v > 127) v = 127;
        c[i] = (int32_t)v;
    }
}

/* Round-to-nearest-even of a double to the nearest bfloat16 value (8 significant
 * bits), done directly on the double so there is no double rounding through
 * float32.  The inter-layer activations of the bf16 nets pass through this.
 * Finite inputs only; bf16 subnormals are handled by the frexp scaling. */
static double round_bf16_one(double x)
{
    if (x == 0.0 || !isfinite(x)) return x;
    int e;
    double m = frexp(x, &e);            /* x = m * 2^e, 0.5 <= |m| < 1 */
    int keep = 8;                       /* significant bits of bf16 */
    const int emin = -125;              /* frexp exponent of the smallest normal (2^-126) */
    if (e < emin) keep -= (emin - e);   /* subnormal range: fewer bits */
    if (keep <= 0) {
        /* below half the smallest subnormal rounds to zero, ties to even (zero) */
        double tiny = ldexp(1.0, -133); /* smallest bf16 subnormal 2^-133 */
        if (fabs(x) > tiny * 0.5) return copysign(tiny, x);
        return copysign(0.0, x);
    }
    double scaled = ldexp(m, keep);     /* |scaled| in [2^(keep-1), 2^keep) */
    double r = nearbyint(scaled);       /* default rounding mode: ties to even */
    return ldexp(r, e - keep);
}

void orc_round_bf16(double* a, long long n)
{
    for (long long i = 0; i < n; ++i) a[i] = round_bf16_one(a[i]);
}

/* 2x2 max pooling, stride 2, floor (a trailing odd row or column is dropped).
 * Not described in the paper; required by the workloads.  1D maps (W == 1)
 * pool over the row axis only. */
void orc_maxpool2_f64(const double* in, long long n_streams, int H, int W, int C, double* out)
{
    const int Ho = H / 2, Wo = (W == 1) ? 1 : W / 2, px = (W == 1) ? 1 : 2;
    for (long long s = 0; s < n_streams; ++s)
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox)
                for (int c = 0; c < C; ++c) {
                    double m = in[(((size_t)s * H + 2 * oy) * W + px * ox) * C + c];
                    for (int dy = 0; dy < 2; ++dy)
                        for (int dx = 0; dx < px; ++dx) {
                            double v = in[(((size_t)s * H + 2 * oy + dy) * W + px * ox + dx) * C + c];
                            if (v > m) m = v;
                        }
                    out[(((size_t)s * Ho + oy) * Wo + ox) * C + c] = m;
                }
}

void orc_maxpool2_i32(const int32_t* in, long long n_streams, int H, int W, int C, int32_t* out)
{
    const int Ho = H / 2, Wo = (W == 1) ? 1 : W / 2, px = (W == 1) ? 1 : 2;
    for (long long s = 0; s < n_streams; ++s)
        for (int oy = 0; oy < Ho; ++oy)
            for (int ox = 0; ox < Wo; ++ox)
                for (int c = 0; c < C; ++c) {
                    int32_t m = in[(((size_t)s * H + 2 * oy) * W + px * ox) * C + c];
                    for (int dy = 0; dy < 2; ++dy)
                        for (int dx = 0; dx < px; ++dx) {
                            int32_t v = in[(((size_t)s * H + 2 * oy + dy) * W + px * ox + dx) * C + c];
                            if (v > m) m = v;
                        }
                    out[(((size_t)s * Ho + oy) * Wo + ox) * C + c] = m;
                }
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
