/*
 * Event-by-event checker (test infrastructure only; tiny inputs).
 *
 * A literal implementation of the stateful neuron of Eq. 2-5: every unit keeps
 * a state variable c, its activation is h = f(c) (Eq. 2), a change of h is
 * sent as an event dh = h(t) - h(t-1) only when it is non-zero (Eq. 3), and a
 * receiving unit adds w * dh to its own state (Eq. 4), which may change its
 * activation and send events further up (Eq. 5 and the sentence after it).
 * Convolutional connectivity: a unit reaches only the kernel-sized
 * neighbourhood above it.
 *
 * It shares no code with idf_oracle.c and exists to pin that oracle: on small
 * nets the final maps produced here, one input component at a time, must equal
 * the layer-by-layer result (the equivalence stated after Eq. 5).
 *
 * Emission policies:
 *   eager    - the paper's: a unit emits the moment its activation changes (one input component at a time).
 *   eager, per segment (eager == 2) - the same rule with all components of a segment delivered before the
 *              layers re-evaluate, one layer after the other: a unit emits h(after the segment) - h(before).
 *   deferred - a unit emits once, when no present or future input can reach
 *              it any more (its row has received its last kernel tap); this
 *              is the policy under which a layer needs only ceil(Kh/stride)
 *              rows of state.
 * Also tracked: per-unit sum of emitted events (telescoping check, Eq. 3+5),
 * event counts per layer, and the number of units that hold state which
 * present or future input can still influence (the quantity the paper's
 * memory claims are about; Fig. 1 prints 7 for its toy net).
 *
 * Units' states are doubles in every numeric mode; integer nets stay exact
 * because all their values are integers below 2^53.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

enum { EVC_CONV = 0, EVC_MAXPOOL2 = 1, EVC_GLOBAL_AVG = 2 };
enum { EVC_F64 = 0, EVC_BF16 = 1, EVC_INT = 2 };

typedef struct { int kind, cin, cout, kh, kw, stride, pad, relu, shift; } evc_layer;

typedef struct {
    int n_layers, mode, eager;
    const evc_layer* L;
    const double* const* w;     /* per layer (NULL for non-conv): [Cout][Kh][Kw][Cin] */
    const double* const* b;     /* per layer or NULL */
    int H[64], W[64], C[64];    /* map sizes; index 0 = input */
    double* c[64];              /* state per layer (index n = layer n, 1-based) */
    double* h[64];              /* current activation per layer; h[0] = input as presented so far */
    double* sum_dh[64];         /* sum of all events a unit has emitted */
    unsigned char* touched[64]; /* unit has received an event or holds a non-zero bias */
    unsigned char* done[64];    /* deferred: unit has emitted */
    long long n_events[64];     /* events emitted by layer n (n = 0: input events) */
    long long n_updates[64];    /* state updates c += w*dh performed in layer n */
    int last_in_row[64];        /* scratch */
} evc_net;

/* bf16 round-to-nearest-even, worked on the double's own bit pattern (add half
 * of the dropped field, plus the kept LSB for ties, then truncate). */
static double evc_bf16(double x)
{
    if (x == 0.0) return x;
    uint64_t u; memcpy(&u, &x, 8);
    /* double: 1 sign, 11 exp, 52 mantissa; bf16 keeps 7 explicit mantissa bits */
    const int drop = 52 - 7;
    uint64_t keep_lsb = (u >> drop) & 1u;
    uint64_t bias = (((uint64_t)1 << (drop - 1)) - 1) + keep_lsb;
    u += bias;                       /* carries into the exponent on overflow, as intended */
    u &= ~((((uint64_t)1) << drop) - 1);
    double r; memcpy(&r, &u, 8);
    return r;                        /* test nets never reach the bf16 subnormal range */
}

static double evc_act(const evc_net* N, int n, double c)
{
    const evc_layer* l = &N->L[n - 1];
    double v = c;
    if (l->relu && v < 0.0) v = 0.0;
    if (N->mode == EVC_BF16) {
        /* rounded only when a later convolution consumes it */
        int feeds_conv = 0;
        for (int k = n + 1; k <= N->n_layers; ++k) feeds_conv |= (N->L[k - 1].kind == EVC_CONV);
        if (feeds_conv) v = evc_bf16(v);
    } else if (N->mode == EVC_INT) {
        if (l->shift > 0) v = floor((v + ldexp(1.0, l->shift - 1)) / ldexp(1.0, l->shift));
        double lo = l->relu ? 0.0 : -127.0;
        if (v < lo) v = lo;
        if (v > 127.0) v = 127.0;
    }
    return v;
}

static void deliver(evc_net* N, int n, int y, int x, int ch, double d);

/* unit (y,x,ch) of layer n re-evaluates its activation and emits if it changed */
static void reevaluate(evc_net* N, int n, int y, int x, int ch)
{
    size_t i = ((size_t)y * N->W[n] + x) * N->C[n] + ch;
    double nh;
    const evc_layer* l = &N->L[n - 1];
    if (l->kind == EVC_CONV) {
        nh = evc_act(N, n, N->c[n][i]);
    } else if (l->kind == EVC_MAXPOOL2) {
        int px = (N->W[n - 1] == 1) ? 1 : 2;
        double m = -INFINITY;
        for (int dy = 0; dy < 2; ++dy)
            for (int dx = 0; dx < px; ++dx) {
                double v = N->h[n - 1][((size_t)(2 * y + dy) * N->W[n - 1] + px * x + dx) * N->C[n - 1] + ch];
                if (v > m) m = v;
            }
        nh = m;
    } else {
        nh = N->c[n][i];
    }
    double d = nh - N->h[n][i];
    if (d != 0.0) {
        N->h[n][i] = nh;
        N->sum_dh[n][i] += d;
        N->n_events[n] += 1;
        if (n < N->n_layers) deliver(N, n + 1, y, x, ch, d);
    }
}

/* Eq. 4: an event d from unit (y,x,ch) of layer n-1 arrives at layer n */
static void deliver(evc_net* N, int n, int y, int x, int ch, double d)
{
    const evc_layer* l = &N->L[n - 1];
    if (l->kind == EVC_CONV) {
        for (int ky = 0; ky < l->kh; ++ky) {
            int ty = y + l->pad - ky;
            if (ty < 0 || ty % l->stride) continue;
            int oy = ty / l->stride;
            if (oy >= N->H[n]) continue;
            const int one_d = (N->W[n - 1] == 1 && l->kw == 1);   /* degenerate x axis: no pad, no stride */
            const int pad_x = one_d ? 0 : l->pad, stride_x = one_d ? 1 : l->stride;
            for (int kx = 0; kx < l->kw; ++kx) {
                int tx = x + pad_x - kx;
                if (tx < 0 || tx % stride_x) continue;
                int ox = tx / stride_x;
                if (ox >= N->W[n]) continue;
                for (int co = 0; co < l->cout; ++co) {
                    size_t i = ((size_t)oy * N->W[n] + ox) * N->C[n] + co;
                    N->c[n][i] += N->w[n - 1][(((size_t)co * l->kh + ky) * l->kw + kx) * l->cin + ch] * d;
                    N->touched[n][i] = 1;
                    N->n_updates[n] += 1;
                    if (N->eager == 1) reevaluate(N, n, oy, ox, co);
                }
            }
        }
    } else if (l->kind == EVC_MAXPOOL2) {
        int px = (N->W[n - 1] == 1) ? 1 : 2;
        int oy = y / 2, ox = x / px;
        if (oy >= N->H[n] || ox >= N->W[n]) return;
        size_t i = ((size_t)oy * N->W[n] + ox) * N->C[n] + ch;
        N->touched[n][i] = 1;
        N->n_updates[n] += 1;
        if (N->eager == 1) reevaluate(N, n, oy, ox, ch);
    } else { /* global average over all positions of a channel */
        size_t i = (size_t)ch;
        N->c[n][i] += d / ((double)N->H[n - 1] * N->W[n - 1]);
        N->touched[n][i] = 1;
        N->n_updates[n] += 1;
        if (N->eager == 1) reevaluate(N, n, 0, 0, ch);
    }
}

/* last input row (clipped to the map) that can influence row oy of layer n */
static int last_input_row(const evc_net* N, int n, int oy)
{
    int r = oy;
    for (int k = n; k >= 1; --k) {
        const evc_layer* l = &N->L[k - 1];
        if (l->kind == EVC_CONV) r = r * l->stride - l->pad + l->kh - 1;
        else if (l->kind == EVC_MAXPOOL2) r = 2 * r + 1;
        else r = N->H[k - 1] - 1;
        if (r > N->H[k - 1] - 1) r = N->H[k - 1] - 1;
        if (r < 0) r = 0;
    }
    return r;
}

/* deferred policy: after input row r has been delivered, finalise (in depth
 * order) every row that can no longer be reached and pass its events on */
static void finalise_ready_rows(evc_net* N, int r_in, int flush, long long* live_peak)
{
    for (int n = 1; n <= N->n_layers; ++n) {
        /* live units right now in layer n (before finalisation = peak of this step) */
        long long live = 0;
        size_t tot = (size_t)N->H[n] * N->W[n] * N->C[n];
        for (size_t i = 0; i < tot; ++i) live += (N->touched[n][i] && !N->done[n][i]);
        if (live > live_peak[n]) live_peak[n] = live;
        for (int oy = 0; oy < N->H[n]; ++oy) {
            int ready = 1;
            if (!flush) {
                /* The stream does not know where the input ends, so a row that waits for
                 * rows below the map (bottom zero padding) completes only at flush: the
                 * test walks down the layers without clipping to the map height. */
                int r = oy;
                for (int k = n; k >= 1; --k) {
                    const evc_layer* l = &N->L[k - 1];
                    if (l->kind == EVC_CONV) r = r * l->stride - l->pad + l->kh - 1;
                    else if (l->kind == EVC_MAXPOOL2) r = 2 * r + 1;
                    else r = 1 << 28;
                }
                if (r > r_in) ready = 0;
            }
            if (!ready) continue;
            for (int x = 0; x < N->W[n]; ++x)
                for (int ch = 0; ch < N->C[n]; ++ch) {
                    size_t i = ((size_t)oy * N->W[n] + x) * N->C[n] + ch;
                    if (N->done[n][i]) continue;
                    N->done[n][i] = 1;
                    reevaluate(N, n, oy, x, ch);   /* emits f(c) - 0 once */
                }
        }
    }
}

/*
 * Run one stream.
 *   input [H][W][C0]; out receives the final activation map of the last layer;
 *   out_sum_dh receives, for the last layer, the sum of emitted events per unit;
 *   stats[0..n_layers]   events emitted per layer (0 = input),
 *   stats2[1..n_layers]  state updates per layer,
 *   live_between[n]      max over steps of (units holding state that future input can still
 *                        influence), counted after each input segment (row),
 *   live_peak[n]         deferred policy: max units allocated at once,
 *   telescoping_err      max over all units of |sum of events - final activation|.
 * Returns 0, or -1 on bad arguments.
 */
/* every unit of layer n re-evaluates once (per-segment eager policy) */
static void reevaluate_layer(evc_net* N, int n)
{
    for (int y = 0; y < N->H[n]; ++y)
        for (int x = 0; x < N->W[n]; ++x)
            for (int ch = 0; ch < N->C[n]; ++ch) reevaluate(N, n, y, x, ch);
}

/*
 * As evc_run, but only the first n_feed rows of the H-row input are presented (the maps are sized for H rows:
 * a stream that does not know yet where its input ends), and after every presented row the activation map of
 * the last layer is copied to steps_out[r] (n_feed maps; may be NULL).  With n_feed == H this is evc_run.
 */
int evc_run_steps(int mode, int eager, int n_layers, const evc_layer* layers,
                  const double* const* weights, const double* const* biases,
                  int H, int W, int C0, const double* input, int n_feed, double* steps_out,
                  double* out, double* out_sum_dh,
                  long long* stats, long long* stats2,
                  long long* live_between, long long* live_peak, double* telescoping_err)
{
    if (n_feed < 0 || n_feed > H) return -1;
    if (n_layers < 1 || n_layers > 62) return -1;
    evc_net N; memset(&N, 0, sizeof N);
    N.n_layers = n_layers; N.mode = mode; N.eager = eager; N.L = layers; N.w = weights; N.b = biases;
    N.H[0] = H; N.W[0] = W; N.C[0] = C0;
    for (int n = 1; n <= n_layers; ++n) {
        const evc_layer* l = &layers[n - 1];
        if (l->kind == EVC_CONV) {
            N.H[n] = (N.H[n - 1] + 2 * l->pad - l->kh) / l->stride + 1;
            N.W[n] = (N.W[n - 1] == 1 && l->kw == 1) ? 1 : (N.W[n - 1] + 2 * l->pad - l->kw) / l->stride + 1;
            N.C[n] = l->cout;
        } else if (l->kind == EVC_MAXPOOL2) {
            N.H[n] = N.H[n - 1] / 2; N.W[n] = (N.W[n - 1] == 1) ? 1 : N.W[n - 1] / 2; N.C[n] = N.C[n - 1];
        } else {
            N.H[n] = 1; N.W[n] = 1; N.C[n] = N.C[n - 1];
        }
        if (N.H[n] < 1 || N.W[n] < 1) return -1;
    }
    for (int n = 0; n <= n_layers; ++n) {
        size_t tot = (size_t)N.H[n] * N.W[n] * N.C[n];
        N.c[n] = (double*)calloc(tot, sizeof(double));
        N.h[n] = (double*)calloc(tot, sizeof(double));
        N.sum_dh[n] = (double*)calloc(tot, sizeof(double));
        N.touched[n] = (unsigned char*)calloc(tot, 1);
        N.done[n] = (unsigned char*)calloc(tot, 1);
        live_between[n] = 0; live_peak[n] = 0;
    }
    /* biases: the state starts at b (a weight from a constant input that is on from the start) */
    for (int n = 1; n <= n_layers; ++n) {
        if (layers[n - 1].kind != EVC_CONV || !biases || !biases[n - 1]) continue;
        size_t pos = (size_t)N.H[n] * N.W[n];
        for (size_t p = 0; p < pos; ++p)
            for (int ch = 0; ch < N.C[n]; ++ch) {
                N.c[n][p * N.C[n] + ch] = biases[n - 1][ch];
                if (biases[n - 1][ch] != 0.0) N.touched[n][p * N.C[n] + ch] = 1;
            }
    }
    if (eager)   /* units whose f(b) is non-zero announce it before any input arrives */
        for (int n = 1; n <= n_layers; ++n) reevaluate_layer(&N, n);

    for (int r = 0; r < n_feed; ++r) {
        /* present the components of this segment one by one; zero components send nothing */
        for (int x = 0; x < W; ++x)
            for (int ch = 0; ch < C0; ++ch) {
                size_t i = ((size_t)r * W + x) * C0 + ch;
                double d = input[i] - N.h[0][i];
                if (d != 0.0) {
                    N.h[0][i] = input[i];
                    N.sum_dh[0][i] += d;
                    N.n_events[0] += 1;
                    deliver(&N, 1, r, x, ch, d);
                }
            }
        if (!eager) finalise_ready_rows(&N, r, 0, live_peak);
        if (eager == 2)   /* the segment is in: the layers re-evaluate one after the other */
            for (int n = 1; n <= n_layers; ++n) reevaluate_layer(&N, n);
        if (steps_out) {
            size_t tot = (size_t)N.H[n_layers] * N.W[n_layers] * N.C[n_layers];
            memcpy(steps_out + (size_t)r * tot, N.h[n_layers], tot * sizeof(double));
        }
        /* units that hold state and that a later segment can still influence */
        for (int n = 1; n <= n_layers; ++n) {
            long long live = 0;
            for (int oy = 0; oy < N.H[n]; ++oy) {
                int can = last_input_row(&N, n, oy) > r;
                if (layers[n - 1].kind == EVC_GLOBAL_AVG) can = 1;
                if (!can) continue;
                for (int x = 0; x < N.W[n]; ++x)
                    for (int ch = 0; ch < N.C[n]; ++ch) {
                        size_t i = ((size_t)oy * N.W[n] + x) * N.C[n] + ch;
                        live += N.touched[n][i] ? 1 : 0;
                    }
            }
            if (live > live_between[n]) live_between[n] = live;
        }
    }
    if (!eager && n_feed == H) finalise_ready_rows(&N, H - 1, 1, live_peak);

    double terr = 0.0;
    for (int n = 0; n <= n_layers; ++n) {
        size_t tot = (size_t)N.H[n] * N.W[n] * N.C[n];
        for (size_t i = 0; i < tot; ++i) {
            double e = fabs(N.sum_dh[n][i] - N.h[n][i]);
            if (e > terr) terr = e;
        }
        stats[n] = N.n_events[n];
        stats2[n] = N.n_updates[n];
    }
    *telescoping_err = terr;
    {
        size_t tot = (size_t)N.H[n_layers] * N.W[n_layers] * N.C[n_layers];
        memcpy(out, N.h[n_layers], tot * sizeof(double));
        if (out_sum_dh) memcpy(out_sum_dh, N.sum_dh[n_layers], tot * sizeof(double));
    }
    for (int n = 0; n <= n_layers; ++n) {
        free(N.c[n]); free(N.h[n]); free(N.sum_dh[n]); free(N.touched[n]); free(N.done[n]);
    }
    return 0;
}

int evc_run(int mode, int eager, int n_layers, const evc_layer* layers,
            const double* const* weights, const double* const* biases,
            int H, int W, int C0, const double* input,
            double* out, double* out_sum_dh,
            long long* stats, long long* stats2,
            long long* live_between, long long* live_peak, double* telescoping_err)
{
    return evc_run_steps(mode, eager, n_layers, layers, weights, biases, H, W, C0, input, H, NULL, out, out_sum_dh,
                         stats, stats2, live_between, live_peak, telescoping_err);
}
