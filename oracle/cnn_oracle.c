/*
 * CPU oracle for the worker side of parameter-server training: the small CNN of
 * the paper's model endnote (two 3x3 convolutions with 16 and 32 filters, each
 * followed by ReLU and 2x2 max pooling; flatten; a 512-unit dense layer with
 * ReLU; 25 % dropout; a 10-unit output layer), its softmax cross-entropy loss,
 * and the gradient of that loss with respect to every parameter.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code with the CUDA path and must
 * never be called from it.  Everything is computed in double precision with
 * direct (non-im2col, non-blocked) loops so that it can be checked against the
 * model description by eye.
 *
 * The paper's endnote fixes only filter counts, layer order, widths and the
 * dropout rate.  The remaining choices (3x3 kernels with zero padding 1,
 * 2x2/stride-2 pooling, 1x28x28 input, channel-major flatten, mean softmax
 * cross-entropy) are the readings recorded in the design notes.
 *
 * Canonical flat parameter layout (floats / doubles, same order for gradients):
 *   conv1.w [16][1][3][3]   at      0
 *   conv1.b [16]            at    144
 *   conv2.w [32][16][3][3]  at    160
 *   conv2.b [32]            at   4768
 *   fc1.w   [512][1568]     at   4800   (out, in; in = c*49 + y*7 + x)
 *   fc1.b   [512]           at 807616
 *   fc2.w   [10][512]       at 808128
 *   fc2.b   [10]            at 813248
 *   total P = 813258
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define IMG 28
#define C1 16
#define H1 14
#define C2 32
#define H2 7
#define FLAT (C2 * H2 * H2) /* 1568 */
#define HID 512
#define NCLS 10

#define OFF_C1W 0
#define OFF_C1B 144
#define OFF_C2W 160
#define OFF_C2B 4768
#define OFF_F1W 4800
#define OFF_F1B 807616
#define OFF_F2W 808128
#define OFF_F2B 813248
#define P_TOTAL 813258

int64_t oracle_param_count(void) { return P_TOTAL; }

/* ------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
 * easy as 1, 2, 3", SC'11): ten rounds; each round multiplies counter words 0
 * and 2 by two fixed 32-bit constants, keeps both halves of the 64-bit
 * products, xors the high halves with the other counter words and the key,
 * and then advances the key by two Weyl constants.
 * ---------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Dropout keep mask for one worker's batch (model endnote: 25 % dropout after
 * the 512-unit layer).  The keying is this project's reading: key = the two
 * halves of `seed`; counter = (q, worker, step low, step high) where the
 * element (sample i, unit j) has linear index e = i*512 + j, q = e / 4, and
 * uses output word e % 4.  An element is kept iff its word >= floor(p * 2^32),
 * an integer comparison, so P(keep) = 1 - p up to 2^-32.
 */
void oracle_dropout_keep(uint64_t seed, uint32_t worker, uint64_t step, int32_t b, double p,
                         uint8_t* keep /* [b*512] */) {
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    double t = floor(p * 4294967296.0);
    uint32_t thresh = t <= 0.0 ? 0u : (t >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)t);
    int64_t n = (int64_t)b * HID;
    for (int64_t q = 0; q * 4 < n; ++q) {
        uint32_t ctr[4] = {(uint32_t)q, worker, (uint32_t)step, (uint32_t)(step >> 32)};
        uint32_t r[4];
        oracle_philox4x32_10(ctr, key, r);
        for (int w = 0; w < 4 && q * 4 + w < n; ++w) keep[q * 4 + w] = (uint8_t)(r[w] >= thresh);
    }
}

/* 3x3 convolution, zero padding 1, stride 1: out[oc][y][x] = b[oc] + sum w*in. */
static void conv3x3(const double* in, int cin, int hw, const double* w, const double* bias,
                    int cout, double* out) {
    for (int oc = 0; oc < cout; ++oc)
        for (int y = 0; y < hw; ++y)
            for (int x = 0; x < hw; ++x) {
                double s = bias[oc];
                for (int ic = 0; ic < cin; ++ic)
                    for (int ky = 0; ky < 3; ++ky)
                        for (int kx = 0; kx < 3; ++kx) {
                            int yy = y + ky - 1, xx = x + kx - 1;
                            if (yy < 0 || yy >= hw || xx < 0 || xx >= hw) continue;
                            s += w[((oc * cin + ic) * 3 + ky) * 3 + kx] * in[(ic * hw + yy) * hw + xx];
                        }
                out[(oc * hw + y) * hw + x] = s;
            }
}

/* Decisions of "ReLU then 2x2/stride-2 max pooling" on pre-activations a: per pooled element the
 * index 0..3 (row-major inside the window) of the first maximum of the rectified values (strict >),
 * or 4 when that maximum is not positive (then no gradient flows through the element). */
static void pool_decide(const double* a, int c, int hw, int* code) {
    int ho = hw / 2;
    for (int ch = 0; ch < c; ++ch)
        for (int y = 0; y < ho; ++y)
            for (int x = 0; x < ho; ++x) {
                double best = 0.0;
                int bi = 0;
                for (int j = 0; j < 4; ++j) {
                    double v = a[(ch * hw + 2 * y + j / 2) * hw + 2 * x + j % 2];
                    double r = v > 0.0 ? v : 0.0;
                    if (j == 0 || r > best) { best = r; bi = j; }
                }
                code[(ch * ho + y) * ho + x] = best > 0.0 ? bi : 4;
            }
}

/* ReLU + max pooling with the decisions given: the pooled value is the pre-activation at the
 * chosen position, or 0 for a dead element. */
static void pool_apply(const double* a, const int* code, int c, int hw, double* pooled) {
    int ho = hw / 2;
    for (int ch = 0; ch < c; ++ch)
        for (int y = 0; y < ho; ++y)
            for (int x = 0; x < ho; ++x) {
                int j = code[(ch * ho + y) * ho + x];
                pooled[(ch * ho + y) * ho + x] =
                    j < 4 ? a[(ch * hw + 2 * y + j / 2) * hw + 2 * x + j % 2] : 0.0;
            }
}

/* Backward of pool_apply: the pooled gradient goes to the chosen position of a live element. */
static void pool_bwd(const double* dpooled, const int* code, int c, int hw, double* da) {
    int ho = hw / 2;
    memset(da, 0, sizeof(double) * (size_t)c * hw * hw);
    for (int ch = 0; ch < c; ++ch)
        for (int y = 0; y < ho; ++y)
            for (int x = 0; x < ho; ++x) {
                int j = code[(ch * ho + y) * ho + x];
                if (j < 4) da[(ch * hw + 2 * y + j / 2) * hw + 2 * x + j % 2] = dpooled[(ch * ho + y) * ho + x];
            }
}

/* ---- operand rounding of a reduced-precision contraction ----------------------------------
 * A tensor-core path rounds the operands of its dense contractions (second convolution, 512-unit
 * layer) to a short mantissa and accumulates exactly enough that the products dominate the error.
 * ReLU signs and pooling winners are integer decisions taken on those rounded results, so the
 * oracle must be able to take them in the same precision.  Rounding modes of an fp32 value:
 *   0  none
 *   1  TF32: 10 explicit mantissa bits, round to nearest, ties away from zero
 *   2  BF16:  7 explicit mantissa bits, round to nearest, ties to even */
static double round_operand(double v, int mode) {
    if (mode == 0) return v;
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    if (mode == 1) u = (u + 0x1000u) & 0xFFFFE000u;
    else u = (u + 0x7FFFu + ((u >> 16) & 1u)) & 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

double oracle_round_operand(double v, int32_t mode) { return round_operand(v, mode); }

/* Which rounding the two reduced-precision contractions use under a given `precision` of the
 * gradient step: 1 = TF32 everywhere; 2 = BF16 operands in the second convolution, TF32 in the
 * 512-unit layer. */
static int conv_rounding(int precision) { return precision == 2 ? 2 : (precision == 1 ? 1 : 0); }
static int dense_rounding(int precision) { return precision != 0 ? 1 : 0; }

/* conv3x3 with both operands rounded in the given mode (0 = plain conv3x3). */
static void conv3x3_rounded(const double* in, int cin, int hw, const double* w, const double* bias,
                            int cout, int precision, double* out) {
    size_t nin = (size_t)cin * hw * hw, nw = (size_t)cout * cin * 9;
    double* inr = malloc(sizeof(double) * nin);
    double* wr = malloc(sizeof(double) * nw);
    for (size_t i = 0; i < nin; ++i) inr[i] = round_operand(in[i], precision);
    for (size_t i = 0; i < nw; ++i) wr[i] = round_operand(w[i], precision);
    conv3x3(inr, cin, hw, wr, bias, cout, out);
    free(inr); free(wr);
}

/* Gradient of conv3x3 with respect to weights and bias (accumulated). */
static void conv3x3_bwd_w(const double* in, int cin, int hw, const double* dout, int cout,
                          double* gw, double* gb) {
    for (int oc = 0; oc < cout; ++oc) {
        double sb = 0.0;
        for (int i = 0; i < hw * hw; ++i) sb += dout[oc * hw * hw + i];
        gb[oc] += sb;
        for (int ic = 0; ic < cin; ++ic)
            for (int ky = 0; ky < 3; ++ky)
                for (int kx = 0; kx < 3; ++kx) {
                    double s = 0.0;
                    for (int y = 0; y < hw; ++y)
                        for (int x = 0; x < hw; ++x) {
                            int yy = y + ky - 1, xx = x + kx - 1;
                            if (yy < 0 || yy >= hw || xx < 0 || xx >= hw) continue;
                            s += dout[(oc * hw + y) * hw + x] * in[(ic * hw + yy) * hw + xx];
                        }
                    gw[((oc * cin + ic) * 3 + ky) * 3 + kx] += s;
                }
    }
}

/* Gradient of conv3x3 with respect to its input. */
static void conv3x3_bwd_x(const double* dout, int cout, int hw, const double* w, int cin,
                          double* din) {
    memset(din, 0, sizeof(double) * (size_t)cin * hw * hw);
    for (int oc = 0; oc < cout; ++oc)
        for (int y = 0; y < hw; ++y)
            for (int x = 0; x < hw; ++x) {
                double g = dout[(oc * hw + y) * hw + x];
                if (g == 0.0) continue;
                for (int ic = 0; ic < cin; ++ic)
                    for (int ky = 0; ky < 3; ++ky)
                        for (int kx = 0; kx < 3; ++kx) {
                            int yy = y + ky - 1, xx = x + kx - 1;
                            if (yy < 0 || yy >= hw || xx < 0 || xx >= hw) continue;
                            din[(ic * hw + yy) * hw + xx] += g * w[((oc * cin + ic) * 3 + ky) * 3 + kx];
                        }
            }
}

/* Optional per-sample intermediates of the exact (double) pass, for tests that ask how far a decision
 * is from flipping.  Nothing here is new arithmetic: every array is a value the step computes anyway.
 * Any pointer may be NULL.  The one input, `flip`, overrides single ReLU decisions of the 512-unit layer (a unit that is
 * switched on passes its pre-activation, whatever its sign, exactly as the backward pass then assumes). */
typedef struct {
    double* p1;      /* [b][16][14][14] pooled output of the first convolution (the second one's input)        */
    double* a2;      /* [b][32][14][14] pre-activations of the second convolution                               */
    double* p2;      /* [b][1568]       pooled output of the second convolution, channel-major flatten          */
    double* u;       /* [b][512]        pre-activations of the 512-unit layer                                   */
    double* dh;      /* [b][512]        gradient of the mean loss w.r.t. the layer's output AFTER its ReLU,     */
                     /*                 dropout applied: a unit that is on contributes dh * p2 to its row       */
    int32_t* code2;  /* [b][1568]       pooling decision of the second convolution that was used (0..3, 4 dead) */
    int32_t* on;     /* [b][512]        ReLU decision of the 512-unit layer that was used                       */
    const uint8_t* flip; /* INPUT, [b][512] or NULL: 1 = take this unit's ReLU decision the other way.  For tests  */
                     /*                 that ask what the exact gradient is under a different, equally valid choice */
                     /*                 at a unit whose pre-activation is within rounding distance of zero           */
} oracle_diag;

/*
 * One worker's gradient step in double precision.
 *   theta  [P]          parameters (canonical layout)
 *   x      [b][28][28]  images
 *   y      [b]          labels 0..9
 *   keep   [b][512]     dropout keep mask (1 = keep), or NULL for no dropout
 *   drop_p              dropout rate; kept activations are scaled by 1/(1-p)
 *   precision           0: every decision (ReLU signs, pooling winners) is taken on the exact
 *                       double-precision values.  1: the decisions are taken the way a TF32
 *                       tensor-core path takes them, on a second forward pass whose second
 *                       convolution and 512-unit layer use TF32-rounded operands (and fp32-stored
 *                       activations); all VALUES are still the exact double-precision ones.
 *                       2: the same, with BF16-rounded operands in the second convolution (the
 *                       512-unit layer stays TF32).
 * Outputs (any may be NULL except grad):
 *   grad   [P]          d(mean loss)/d(theta)
 *   loss                mean over the batch of logsumexp(z) - z[y]
 *   argmax [b]          lowest index of the maximal logit
 *   logits [b][10]
 *   diag                optional intermediates of the exact pass (see oracle_diag), or NULL
 * Returns 0, or -1 on a bad argument (label out of range, b <= 0).
 */
int32_t oracle_grad_step_f64_diag(const double* theta, const double* x, const int32_t* y, int32_t b,
                                  const uint8_t* keep, double drop_p, int32_t precision, double* grad,
                                  double* loss, int32_t* argmax, double* logits, const oracle_diag* diag) {
    if (b <= 0 || !theta || !x || !y || !grad) return -1;
    for (int i = 0; i < b; ++i)
        if (y[i] < 0 || y[i] >= NCLS) return -1;
    const double* c1w = theta + OFF_C1W; const double* c1b = theta + OFF_C1B;
    const double* c2w = theta + OFF_C2W; const double* c2b = theta + OFF_C2B;
    const double* f1w = theta + OFF_F1W; const double* f1b = theta + OFF_F1B;
    const double* f2w = theta + OFF_F2W; const double* f2b = theta + OFF_F2B;
    double scale = keep ? 1.0 / (1.0 - drop_p) : 1.0;

    size_t na1 = (size_t)C1 * IMG * IMG, np1 = (size_t)C1 * H1 * H1;
    size_t na2 = (size_t)C2 * H1 * H1, np2 = FLAT;
    double* a1 = malloc(sizeof(double) * na1); double* da1 = malloc(sizeof(double) * na1);
    double* p1 = malloc(sizeof(double) * np1); double* dp1 = malloc(sizeof(double) * np1);
    double* a2 = malloc(sizeof(double) * na2); double* da2 = malloc(sizeof(double) * na2);
    double* p2 = malloc(sizeof(double) * np2); double* dp2 = malloc(sizeof(double) * np2);
    int* i1 = malloc(sizeof(int) * np1); int* i2 = malloc(sizeof(int) * np2);
    double* p1q = malloc(sizeof(double) * np1); double* a2q = malloc(sizeof(double) * na2);
    double* p2q = malloc(sizeof(double) * np2);
    double u[HID], d[HID], du[HID], z[NCLS], dz[NCLS];
    int on[HID];

    memset(grad, 0, sizeof(double) * P_TOTAL);
    double loss_sum = 0.0;
    for (int i = 0; i < b; ++i) {
        const double* xi = x + (size_t)i * IMG * IMG;
        /* forward */
        conv3x3(xi, 1, IMG, c1w, c1b, C1, a1);
        pool_decide(a1, C1, IMG, i1);            /* the first convolution is exact in every path */
        pool_apply(a1, i1, C1, IMG, p1);
        conv3x3(p1, C1, H1, c2w, c2b, C2, a2);
        if (precision == 0) {
            pool_decide(a2, C2, H1, i2);
        } else {
            /* decision pass in the kernel's precision: activations are stored as fp32 there */
            for (size_t k = 0; k < np1; ++k) p1q[k] = (double)(float)p1[k];
            conv3x3_rounded(p1q, C1, H1, c2w, c2b, C2, conv_rounding(precision), a2q);
            pool_decide(a2q, C2, H1, i2);
            pool_apply(a2q, i2, C2, H1, p2q);
            for (size_t k = 0; k < np2; ++k) p2q[k] = round_operand((double)(float)p2q[k], dense_rounding(precision));
        }
        pool_apply(a2, i2, C2, H1, p2); /* p2 is already the channel-major flatten */
        if (diag) {
            if (diag->p1) memcpy(diag->p1 + (size_t)i * np1, p1, sizeof(double) * np1);
            if (diag->a2) memcpy(diag->a2 + (size_t)i * na2, a2, sizeof(double) * na2);
            if (diag->p2) memcpy(diag->p2 + (size_t)i * np2, p2, sizeof(double) * np2);
            if (diag->code2) for (size_t k = 0; k < np2; ++k) diag->code2[(size_t)i * np2 + k] = i2[k];
        }
        for (int j = 0; j < HID; ++j) {
            double s = f1b[j];
            for (int k = 0; k < FLAT; ++k) s += f1w[(size_t)j * FLAT + k] * p2[k];
            u[j] = s;
            if (precision == 0) {
                on[j] = s > 0.0;
            } else {
                double sq = f1b[j];
                for (int k = 0; k < FLAT; ++k) sq += round_operand(f1w[(size_t)j * FLAT + k], dense_rounding(precision)) * p2q[k];
                on[j] = sq > 0.0;
            }
            if (diag && diag->flip && diag->flip[(size_t)i * HID + j]) on[j] = !on[j];
            double h = on[j] ? s : 0.0;
            int kept = keep ? keep[(size_t)i * HID + j] : 1;
            d[j] = kept ? h * scale : 0.0;
        }
        double zmax = -INFINITY;
        int am = 0;
        for (int c = 0; c < NCLS; ++c) {
            double s = f2b[c];
            for (int j = 0; j < HID; ++j) s += f2w[c * HID + j] * d[j];
            z[c] = s;
            if (s > zmax) { zmax = s; am = c; }
        }
        double se = 0.0;
        for (int c = 0; c < NCLS; ++c) se += exp(z[c] - zmax);
        double lse = zmax + log(se);
        loss_sum += lse - z[y[i]];
        if (argmax) argmax[i] = am;
        if (logits) memcpy(logits + (size_t)i * NCLS, z, sizeof(z));
        /* backward of the mean loss */
        for (int c = 0; c < NCLS; ++c) dz[c] = (exp(z[c] - lse) - (c == y[i] ? 1.0 : 0.0)) / b;
        for (int c = 0; c < NCLS; ++c) {
            grad[OFF_F2B + c] += dz[c];
            for (int j = 0; j < HID; ++j) grad[OFF_F2W + c * HID + j] += dz[c] * d[j];
        }
        for (int j = 0; j < HID; ++j) {
            double s = 0.0;
            for (int c = 0; c < NCLS; ++c) s += f2w[c * HID + j] * dz[c];
            int kept = keep ? keep[(size_t)i * HID + j] : 1;
            double dh = kept ? s * scale : 0.0;
            du[j] = on[j] ? dh : 0.0;
            if (diag && diag->dh) diag->dh[(size_t)i * HID + j] = dh;
            if (diag && diag->u) diag->u[(size_t)i * HID + j] = u[j];
            if (diag && diag->on) diag->on[(size_t)i * HID + j] = on[j];
        }
        memset(dp2, 0, sizeof(double) * np2);
        for (int j = 0; j < HID; ++j) {
            double g = du[j];
            grad[OFF_F1B + j] += g;
            if (g == 0.0) continue;
            for (int k = 0; k < FLAT; ++k) {
                grad[OFF_F1W + (size_t)j * FLAT + k] += g * p2[k];
                dp2[k] += g * f1w[(size_t)j * FLAT + k];
            }
        }
        pool_bwd(dp2, i2, C2, H1, da2);
        conv3x3_bwd_w(p1, C1, H1, da2, C2, grad + OFF_C2W, grad + OFF_C2B);
        conv3x3_bwd_x(da2, C2, H1, c2w, C1, dp1);
        pool_bwd(dp1, i1, C1, IMG, da1);
        conv3x3_bwd_w(xi, 1, IMG, da1, C1, grad + OFF_C1W, grad + OFF_C1B);
    }
    if (loss) *loss = loss_sum / b;
    free(a1); free(da1); free(p1); free(dp1); free(a2); free(da2); free(p2); free(dp2);
    free(i1); free(i2); free(p1q); free(a2q); free(p2q);
    return 0;
}

int32_t oracle_grad_step_f64(const double* theta, const double* x, const int32_t* y, int32_t b,
                             const uint8_t* keep, double drop_p, int32_t precision, double* grad,
                             double* loss, int32_t* argmax, double* logits) {
    return oracle_grad_step_f64_diag(theta, x, y, b, keep, drop_p, precision, grad, loss, argmax, logits, NULL);
}

/*
 * W workers, each with its own fp32 weight snapshot, fp32 images and Philox
 * dropout mask keyed by (seed, worker id, step).  Inputs are widened to double;
 * results stay in double (the caller rounds where the interface is fp32).
 *   thetas     [W] pointers to P floats (workers may share a pointer)
 *   worker_ids [W] logical worker ids used in the dropout key
 *   x [W][b][28][28], y [W][b]
 *   grads [W][P], loss [W], argmax [W][b], logits [W][b][10] (logits may be NULL)
 * Workers are independent, so they are distributed over OpenMP threads when
 * compiled with -fopenmp; the arithmetic per worker is unchanged.
 */
int32_t oracle_workers_grad_step(int32_t W, int32_t b, const float* const* thetas,
                                 const int32_t* worker_ids, const float* x, const int32_t* y,
                                 uint64_t seed, uint64_t step, double drop_p, int32_t precision,
                                 double* grads, double* loss, int32_t* argmax, double* logits) {
    if (W <= 0 || b <= 0) return -1;
    int32_t rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int w = 0; w < W; ++w) {
        double* th = malloc(sizeof(double) * P_TOTAL);
        double* xd = malloc(sizeof(double) * (size_t)b * IMG * IMG);
        uint8_t* keep = malloc((size_t)b * HID);
        for (int64_t i = 0; i < P_TOTAL; ++i) th[i] = (double)thetas[w][i];
        for (int64_t i = 0; i < (int64_t)b * IMG * IMG; ++i) xd[i] = (double)x[(size_t)w * b * IMG * IMG + i];
        const uint8_t* kp = NULL;
        if (drop_p > 0.0) {
            oracle_dropout_keep(seed, (uint32_t)worker_ids[w], step, b, drop_p, keep);
            kp = keep;
        }
        int32_t r = oracle_grad_step_f64(th, xd, y + (size_t)w * b, b, kp, drop_p, precision,
                                         grads + (size_t)w * P_TOTAL, loss ? loss + w : NULL,
                                         argmax ? argmax + (size_t)w * b : NULL,
                                         logits ? logits + (size_t)w * b * NCLS : NULL);
        if (r != 0) {
#pragma omp atomic write
            rc = r;
        }
        free(th); free(xd); free(keep);
    }
    return rc;
}

#ifdef _OPENMP
#include <omp.h>
int32_t oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int32_t oracle_num_threads(void) { return 1; }
#endif
