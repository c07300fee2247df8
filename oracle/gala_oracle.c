/*
 * GALA-A2C oracle: plain, slow, fp64 CPU arithmetic for the learner step of
 * "Gossip-based Actor-Learner Architectures" (arXiv 1906.04585).
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
 * checked against something written straight from the paper.  Only the test
 * suite, the smoke check and the CPU-baseline leg of the benchmark may call
 * it; the product path never does.  It shares no code, header, table or
 * constant with the CUDA sources.
 *
 * Everything is double precision; one loop nest per definition, no blocking,
 * no lowering of convolutions to matrix products, no fusion.
 *
 * What follows which passage of the paper:
 *   orc_returns      n-step return G_t (Sec. 2, text after Eq. 1; Algorithm 1,
 *                    "compute returns and advantages" step)
 *   orc_a2c_loss     TD loss (Eq. 1), policy gradient with baseline (Eq. 2),
 *                    entropy term (Eq. 3), batched mean (Eq. 4)
 *   orc_forward /    the policy/value network of Appendix C.2 ("3 conv layers
 *   orc_backward     and one hidden layer, linear policy and critic outputs")
 *   orc_clip_coef    "Clip global gradient norm" row of Table 2
 *   orc_rmsprop      RMSProp rows of Table 2 (momentum 0)
 *   orc_mix          gossip step of Algorithm 1 with the equal-neighbour
 *                    weights of its footnote; matrix form Eq. 7
 *   orc_sample       "take actions according to pi" (Algorithm 1, acting step)
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_CONV 4
#define ORC_MAX_HID 4
#define ORC_MAX_LAYERS (ORC_MAX_CONV + ORC_MAX_HID)

/* Network description.  Trunk = n_conv VALID convolutions (square kernel,
 * NHWC input, weights [cout][kh][kw][cin]) followed by n_hidden dense layers
 * (weights [out][in]); every trunk layer is followed by the activation `act`
 * (0 = ReLU, 1 = tanh).  Heads: policy W[A][H], b[A]; value W[1][H], b[1].
 * Flat parameter order: for each trunk layer W then b; then policy W, b;
 * then value W, b. */
typedef struct {
    int n_conv;
    int in_h, in_w, in_c;
    int ck[ORC_MAX_CONV], cs[ORC_MAX_CONV], cc[ORC_MAX_CONV];
    int n_hidden;
    int hidden[ORC_MAX_HID];
    int act;
    int n_actions;
    double in_scale; /* observation multiplier (1/255 for byte frames) */
    /* Reduced-precision operand emulation ("bf16 GEMMs, fp32 params"): when set, every trunk
     * layer's output activation and every dL/d(pre-activation) is rounded to bfloat16 (nearest
     * even), as a kernel that stores them in bf16 would; sums stay exact (double).  The caller
     * rounds the trunk weights itself.  0 = exact arithmetic throughout. */
    int round_bf16;
    /* 1: every pre-activation sum of the trunk is formed in float32, term after term in index order, instead of
     * exactly.  Not the method: a second, equally valid evaluation of the rounded network, used to measure how far
     * two implementations that differ only in summation precision drift apart (stored bf16 values one unit in the
     * last place apart, ReLU gates that fall the other way).  Only meaningful with round_bf16. */
    int sum_f32;
} orc_net;

typedef struct {
    int conv; /* 1 = convolution, 0 = dense */
    int ih, iw, ic, k, s, oh, ow, oc;
    long in_size, out_size;
    long w_off, b_off;
} orc_layer;

static int build_layers(const orc_net *net, orc_layer *L, long *pi_w, long *pi_b, long *v_w,
                        long *v_b, long *d_total) {
    int nl = 0;
    long off = 0;
    int h = net->in_h, w = net->in_w, c = net->in_c;
    for (int i = 0; i < net->n_conv; i++) {
        orc_layer *l = &L[nl++];
        l->conv = 1;
        l->ih = h; l->iw = w; l->ic = c;
        l->k = net->ck[i]; l->s = net->cs[i]; l->oc = net->cc[i];
        l->oh = (h - l->k) / l->s + 1;
        l->ow = (w - l->k) / l->s + 1;
        l->in_size = (long)h * w * c;
        l->out_size = (long)l->oh * l->ow * l->oc;
        l->w_off = off; off += (long)l->oc * l->k * l->k * c;
        l->b_off = off; off += l->oc;
        h = l->oh; w = l->ow; c = l->oc;
    }
    long feat = (long)h * w * c;
    for (int i = 0; i < net->n_hidden; i++) {
        orc_layer *l = &L[nl++];
        l->conv = 0;
        l->ih = l->iw = 1; l->ic = (int)feat; l->k = l->s = 1;
        l->oh = l->ow = 1; l->oc = net->hidden[i];
        l->in_size = feat; l->out_size = net->hidden[i];
        l->w_off = off; off += feat * net->hidden[i];
        l->b_off = off; off += net->hidden[i];
        feat = net->hidden[i];
    }
    *pi_w = off; off += feat * net->n_actions;
    *pi_b = off; off += net->n_actions;
    *v_w = off; off += feat;
    *v_b = off; off += 1;
    *d_total = off;
    return nl;
}

long orc_param_count(const orc_net *net) {
    orc_layer L[ORC_MAX_LAYERS];
    long a, b, c, d, tot;
    build_layers(net, L, &a, &b, &c, &d, &tot);
    return tot;
}

/* Offsets of every tensor in the flat vector: out[2*i], out[2*i+1] = W, b
 * offsets of trunk layer i; then policy W, b; value W, b; returns the number
 * of trunk layers. */
int orc_param_offsets(const orc_net *net, long *out) {
    orc_layer L[ORC_MAX_LAYERS];
    long a, b, c, d, tot;
    int nl = build_layers(net, L, &a, &b, &c, &d, &tot);
    for (int i = 0; i < nl; i++) { out[2 * i] = L[i].w_off; out[2 * i + 1] = L[i].b_off; }
    out[2 * nl] = a; out[2 * nl + 1] = b; out[2 * nl + 2] = c; out[2 * nl + 3] = d;
    return nl;
}

/* Round to bfloat16 (8 significant bits, nearest, ties to even), via float32. */
double orc_round_bf16(double v) {
    float f = (float)v;
    unsigned int u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return (double)f; /* inf / nan unchanged */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

static double act_fn(int act, double z) { return act == 0 ? (z > 0.0 ? z : 0.0) : tanh(z); }
/* derivative expressed through the layer OUTPUT a = act(z) */
static double act_grad(int act, double a) { return act == 0 ? (a > 0.0 ? 1.0 : 0.0) : 1.0 - a * a; }

/* One trunk layer, one sample: y = act(W * x + b). */
static void layer_forward(const orc_layer *l, int act, int rnd, int f32, const double *p, const double *x, double *y) {
    const double *W = p + l->w_off, *b = p + l->b_off;
    if (!l->conv) {
        for (int o = 0; o < l->oc; o++) {
            double acc = b[o];
            const double *w = W + (long)o * l->in_size;
            if (f32) {
                float a = (float)b[o];
                for (long i = 0; i < l->in_size; i++) a += (float)w[i] * (float)x[i];
                acc = (double)a;
            } else {
                for (long i = 0; i < l->in_size; i++) acc += w[i] * x[i];
            }
            y[o] = act_fn(act, acc);
            if (rnd) y[o] = orc_round_bf16(y[o]);
        }
        return;
    }
    for (int oy = 0; oy < l->oh; oy++)
        for (int ox = 0; ox < l->ow; ox++)
            for (int o = 0; o < l->oc; o++) {
                double acc = b[o];
                float accf = (float)b[o];
                for (int ky = 0; ky < l->k; ky++)
                    for (int kx = 0; kx < l->k; kx++) {
                        const double *xi = x + ((long)(oy * l->s + ky) * l->iw + (ox * l->s + kx)) * l->ic;
                        const double *w = W + (((long)o * l->k + ky) * l->k + kx) * l->ic;
                        if (f32) for (int c = 0; c < l->ic; c++) accf += (float)w[c] * (float)xi[c];
                        else for (int c = 0; c < l->ic; c++) acc += w[c] * xi[c];
                    }
                if (f32) acc = (double)accf;
                double a = act_fn(act, acc);
                y[((long)oy * l->ow + ox) * l->oc + o] = rnd ? orc_round_bf16(a) : a;
            }
}

/* One trunk layer, one sample, backward.  dy is dL/d(output); it is turned
 * into dL/d(pre-activation) in place.  Accumulates into g (W and b), writes
 * dx (may be NULL for the first layer). */
static void layer_backward(const orc_layer *l, int act, int rnd, const double *p, const double *x,
                           const double *y, double *dy, double *g, double *dx) {
    const double *W = p + l->w_off;
    double *gW = g + l->w_off, *gb = g + l->b_off;
    for (long i = 0; i < l->out_size; i++) {
        dy[i] *= act_grad(act, y[i]);
        if (rnd) dy[i] = orc_round_bf16(dy[i]);
    }
    if (dx) memset(dx, 0, sizeof(double) * (size_t)l->in_size);
    if (!l->conv) {
        for (int o = 0; o < l->oc; o++) {
            double d = dy[o];
            gb[o] += d;
            double *gw = gW + (long)o * l->in_size;
            const double *w = W + (long)o * l->in_size;
            for (long i = 0; i < l->in_size; i++) gw[i] += d * x[i];
            if (dx) for (long i = 0; i < l->in_size; i++) dx[i] += d * w[i];
        }
        return;
    }
    for (int oy = 0; oy < l->oh; oy++)
        for (int ox = 0; ox < l->ow; ox++)
            for (int o = 0; o < l->oc; o++) {
                double d = dy[((long)oy * l->ow + ox) * l->oc + o];
                gb[o] += d;
                for (int ky = 0; ky < l->k; ky++)
                    for (int kx = 0; kx < l->k; kx++) {
                        long xo = ((long)(oy * l->s + ky) * l->iw + (ox * l->s + kx)) * l->ic;
                        long wo = (((long)o * l->k + ky) * l->k + kx) * l->ic;
                        for (int c = 0; c < l->ic; c++) gW[wo + c] += d * x[xo + c];
                        if (dx) for (int c = 0; c < l->ic; c++) dx[xo + c] += d * W[wo + c];
                    }
            }
}

static long max_act_size(const orc_layer *L, int nl) {
    long m = L[0].in_size;
    for (int i = 0; i < nl; i++) if (L[i].out_size > m) m = L[i].out_size;
    return m;
}

/* Forward pass on B observations obs[B][in_size] (raw values, scaled here by
 * in_scale).  Outputs logits[B][A], values[B].  If layer_out != NULL, also
 * copies the post-activation output of trunk layer `which_layer` of every
 * sample to layer_out[B][out_size]. */
int orc_forward(const orc_net *net, const double *params, const double *obs, int B,
                double *logits, double *values, int which_layer, double *layer_out) {
    orc_layer L[ORC_MAX_LAYERS];
    long pw, pb, vw, vb, d;
    int nl = build_layers(net, L, &pw, &pb, &vw, &vb, &d);
    if (nl == 0) return -1;
    long m = max_act_size(L, nl);
    double *a0 = (double *)malloc(sizeof(double) * (size_t)m);
    double *a1 = (double *)malloc(sizeof(double) * (size_t)m);
    if (!a0 || !a1) { free(a0); free(a1); return -2; }
    int A = net->n_actions;
    for (int s = 0; s < B; s++) {
        const double *o = obs + (long)s * L[0].in_size;
        for (long i = 0; i < L[0].in_size; i++) a0[i] = o[i] * net->in_scale;
        double *x = a0, *y = a1;
        for (int li = 0; li < nl; li++) {
            layer_forward(&L[li], net->act, net->round_bf16, net->sum_f32, params, x, y);
            if (layer_out && li == which_layer)
                memcpy(layer_out + (long)s * L[li].out_size, y, sizeof(double) * (size_t)L[li].out_size);
            double *t = x; x = y; y = t;
        }
        long H = L[nl - 1].out_size;
        for (int k = 0; k < A; k++) {
            double acc = params[pb + k];
            for (long j = 0; j < H; j++) acc += params[pw + (long)k * H + j] * x[j];
            if (logits) logits[(long)s * A + k] = acc;
        }
        double acc = params[vb];
        for (long j = 0; j < H; j++) acc += params[vw + j] * x[j];
        if (values) values[s] = acc;
    }
    free(a0); free(a1);
    return 0;
}

/* Backward pass: given dL/dlogits[B][A] and dL/dvalues[B], ACCUMULATES
 * dL/dparams into grad[d] (caller zeroes it).  The forward activations are
 * recomputed sample by sample. */
int orc_backward(const orc_net *net, const double *params, const double *obs, int B,
                 const double *dlogits, const double *dvalues, double *grad) {
    orc_layer L[ORC_MAX_LAYERS];
    long pw, pb, vw, vb, d;
    int nl = build_layers(net, L, &pw, &pb, &vw, &vb, &d);
    if (nl == 0) return -1;
    int A = net->n_actions;
    double *acts[ORC_MAX_LAYERS + 1];
    double *da, *db;
    long m = max_act_size(L, nl);
    acts[0] = (double *)malloc(sizeof(double) * (size_t)L[0].in_size);
    for (int li = 0; li < nl; li++) acts[li + 1] = (double *)malloc(sizeof(double) * (size_t)L[li].out_size);
    da = (double *)malloc(sizeof(double) * (size_t)m);
    db = (double *)malloc(sizeof(double) * (size_t)m);
    for (int s = 0; s < B; s++) {
        const double *o = obs + (long)s * L[0].in_size;
        for (long i = 0; i < L[0].in_size; i++) acts[0][i] = o[i] * net->in_scale;
        for (int li = 0; li < nl; li++) layer_forward(&L[li], net->act, net->round_bf16, net->sum_f32, params, acts[li], acts[li + 1]);
        long H = L[nl - 1].out_size;
        const double *h = acts[nl];
        /* heads */
        for (long j = 0; j < H; j++) da[j] = 0.0;
        for (int k = 0; k < A; k++) {
            double dz = dlogits[(long)s * A + k];
            grad[pb + k] += dz;
            for (long j = 0; j < H; j++) {
                grad[pw + (long)k * H + j] += dz * h[j];
                da[j] += dz * params[pw + (long)k * H + j];
            }
        }
        double dv = dvalues[s];
        grad[vb] += dv;
        for (long j = 0; j < H; j++) {
            grad[vw + j] += dv * h[j];
            da[j] += dv * params[vw + j];
        }
        /* trunk */
        double *dy = da, *dx = db;
        for (int li = nl - 1; li >= 0; li--) {
            layer_backward(&L[li], net->act, net->round_bf16, params, acts[li], acts[li + 1], dy, grad, li > 0 ? dx : NULL);
            double *t = dy; dy = dx; dx = t;
        }
    }
    for (int li = 0; li <= nl; li++) free(acts[li]);
    free(da); free(db);
    return 0;
}

/* n-step returns truncated at the end of the rollout, with episode ends:
 * G_T = V(s_T);  G_t = r_t + gamma * (1 - done_t) * G_{t+1},  t = T-1 .. 0.
 * Without dones this is sum_{i<T-t} gamma^i r_{t+i} + gamma^{T-t} V(s_T). */
void orc_returns(int T, int E, double gamma, const double *r, const unsigned char *done,
                 const double *v_boot, double *G) {
    for (int e = 0; e < E; e++) {
        double g = v_boot[e];
        for (int t = T - 1; t >= 0; t--) {
            g = r[(long)t * E + e] + gamma * (done[(long)t * E + e] ? 0.0 : 1.0) * g;
            G[(long)t * E + e] = g;
        }
    }
}

/* A2C objective over S samples and its derivative w.r.t. logits and values.
 *   L = mean_s[ -log pi(a_s|s) * Adv_s - eta * H(pi_s) ] + c_v * mean_s[(G_s - V_s)^2]
 * with H = -sum_a pi log pi; Adv and G are constants.
 * losses[0] = policy term, [1] = mean squared TD error (without c_v),
 * [2] = mean entropy, [3] = total L. */
void orc_a2c_loss(int S, int A, const double *logits, const int *actions, const double *adv,
                  const double *G, const double *V, double eta, double c_v, double *dlogits,
                  double *dV, double *losses) {
    double lp = 0.0, lv = 0.0, le = 0.0;
    double *pi = (double *)malloc(sizeof(double) * (size_t)A);
    double *lg = (double *)malloc(sizeof(double) * (size_t)A);
    for (int s = 0; s < S; s++) {
        const double *z = logits + (long)s * A;
        double mx = z[0];
        for (int k = 1; k < A; k++) if (z[k] > mx) mx = z[k];
        double sum = 0.0;
        for (int k = 0; k < A; k++) sum += exp(z[k] - mx);
        double lse = mx + log(sum);
        double H = 0.0;
        for (int k = 0; k < A; k++) { lg[k] = z[k] - lse; pi[k] = exp(lg[k]); H -= pi[k] * lg[k]; }
        int a = actions[s];
        lp += -lg[a] * adv[s];
        le += H;
        lv += (G[s] - V[s]) * (G[s] - V[s]);
        if (dlogits)
            for (int k = 0; k < A; k++) {
                /* d(-log pi_a)/dz_k = pi_k - [k == a];  d(-H)/dz_k = pi_k (log pi_k + H) */
                double d = adv[s] * (pi[k] - (k == a ? 1.0 : 0.0)) + eta * pi[k] * (lg[k] + H);
                dlogits[(long)s * A + k] = d / S;
            }
        if (dV) dV[s] = 2.0 * c_v * (V[s] - G[s]) / S;
    }
    free(pi); free(lg);
    if (losses) {
        losses[0] = lp / S; losses[1] = lv / S; losses[2] = le / S;
        losses[3] = lp / S - eta * le / S + c_v * lv / S;
    }
}

/* Global-norm clip coefficient: min(1, max_norm / (||g||_2 + 1e-6));
 * max_norm <= 0 switches clipping off.  Writes ||g||_2 to *norm_out. */
double orc_clip_coef(long d, const double *g, double max_norm, double *norm_out) {
    double ss = 0.0;
    for (long i = 0; i < d; i++) ss += g[i] * g[i];
    double nrm = sqrt(ss);
    if (norm_out) *norm_out = nrm;
    if (max_norm <= 0.0) return 1.0;
    double c = max_norm / (nrm + 1e-6);
    return c < 1.0 ? c : 1.0;
}

/* RMSProp without momentum, epsilon outside the root:
 *   v <- alpha v + (1 - alpha) (c g)^2 ;  y <- x - lr (c g) / (sqrt(v) + eps). */
void orc_rmsprop(long d, const double *x, const double *g, double *v, double clip, double lr,
                 double alpha, double eps, double *y) {
    for (long i = 0; i < d; i++) {
        double gi = clip * g[i];
        v[i] = alpha * v[i] + (1.0 - alpha) * gi * gi;
        y[i] = x[i] - lr * gi / (sqrt(v[i]) + eps);
    }
}

/* Equal-neighbour average: out = (own + sum_j msgs[j]) / (1 + p). */
void orc_mix(long d, const double *own, int p, const double *const *msgs, double *out) {
    double w = 1.0 / (1.0 + p);
    for (long i = 0; i < d; i++) {
        double acc = own[i];
        for (int j = 0; j < p; j++) acc += msgs[j][i];
        out[i] = acc * w;
    }
}

/* Inverse-CDF draw from softmax(z): smallest k with sum_{j<=k} pi_j > u,
 * clamped to A-1. */
int orc_sample(int A, const double *z, double u) {
    double mx = z[0];
    for (int k = 1; k < A; k++) if (z[k] > mx) mx = z[k];
    double sum = 0.0;
    for (int k = 0; k < A; k++) sum += exp(z[k] - mx);
    double cdf = 0.0;
    for (int k = 0; k < A; k++) {
        cdf += exp(z[k] - mx) / sum;
        if (cdf > u) return k;
    }
    return A - 1;
}
