/*
 * DeepPoly oracle: TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, float64 CPU implementation of the DeepPoly certifier as the
 * paper's DeepPoly specification (Appendix C, listing "DeepPoly") defines it,
 * neuron by neuron.  Only tests, the smoke check and the benchmark's CPU
 * baseline leg may build or call this file.  It shares no code, header, table
 * or helper with the CUDA library.
 *
 * What follows which passage (Appendix C, DeepPoly listing, unless noted):
 *   - input box: the abstract shape of an input neuron is its concrete
 *     interval [l,u] (Section 2, "Concrete Bounds"); an L-infinity ball of
 *     radius eps around a centre, intersected with the clip range.
 *   - Affine transformer: L = U = prev.dot(weight) + bias, and
 *     l = backsubs_lower(L), u = backsubs_upper(U).
 *   - backsubs_*: traverse backward, highest layer first (priority2 =
 *     -layer), never stopping early (stop_traverse = false), replacing every
 *     (neuron, coefficient) pair with replace_lower / replace_upper; then
 *     map(simplify_lower / simplify_upper) against concrete bounds.
 *   - replace_lower(n,c) = c >= 0 ? c*n[L] : c*n[U]   (upper: swapped)
 *   - simplify_lower(n,c) = c >= 0 ? c*n[l] : c*n[u]  (upper: swapped)
 *   - Relu transformer: l = relu(prev[l]), u = relu(prev[u]),
 *     L = relu_n(prev) = (l+u >= 0 ? prev : 0),
 *     U = compute_upper(prev) = l >= 0 ? prev
 *                             : u <= 0 ? 0
 *                             : u/(u-l) * prev - u*l/(u-l).
 *
 * Readings taken where the paper is silent:
 *   - the traversal ends when the expression is over input neurons (they
 *     have no L/U), and simplify_* then uses the box;
 *   - ReLU and Affine are separate layers, so one traversal round replaces
 *     all neurons of the highest remaining layer;
 *   - a back-substituted bound is NOT intersected with any other bound;
 *   - conv layers are cross-correlations with zero padding,
 *     out = floor((in + 2*pad - k)/stride) + 1, flattened (c,h,w) row-major;
 *   - the three sign tests of the Relu transformer are taken on l and u
 *     rounded to binary32 and (for l+u) added in binary32 when
 *     decision_fp32 != 0, so that exact ties resolve as in a binary32
 *     implementation; with decision_fp32 == 0 they are taken in float64.
 *     The slopes and intercepts are always computed in float64 from the
 *     float64 l and u.
 *
 * Parity with the paper's own executables is unpinned (they are not
 * available); the pins are the tests under tests/ marked "not gpu".
 *
 * Branch codes per hidden (ReLU) neuron:
 *   0 = stable inactive (u <= 0), 1 = stable active (l >= 0),
 *   2 = unstable with lower slope 0, 3 = unstable with lower slope 1.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int kind;        /* 0 = fully connected, 1 = conv2d                       */
    int relu_after;  /* 1 = a ReLU layer follows this affine layer            */
    int in_features, out_features;              /* FC: weight [out][in]      */
    int c_in, h_in, w_in, c_out, kh, kw, stride, pad; /* conv: [co][ci][kh][kw] */
    const float *weight;
    const float *bias;
} oracle_layer_t;

static int conv_out(int in, int k, int s, int p) { return (in + 2 * p - k) / s + 1; }

static int layer_n_in(const oracle_layer_t *L)
{
    return L->kind == 0 ? L->in_features : L->c_in * L->h_in * L->w_in;
}

static int layer_n_out(const oracle_layer_t *L)
{
    if (L->kind == 0) return L->out_features;
    return L->c_out * conv_out(L->h_in, L->kh, L->stride, L->pad) *
           conv_out(L->w_in, L->kw, L->stride, L->pad);
}

/* The polyhedral expression of affine neuron i over the layer's inputs:
 * coef = row i of the layer's linear map, *d = its bias
 * ("prev.dot(curr[weight]) + curr[bias]").                                   */
static void affine_row(const oracle_layer_t *L, int i, double *coef, double *d)
{
    int n_in = layer_n_in(L);
    if (L->kind == 0) {
        for (int s = 0; s < n_in; ++s) coef[s] = (double)L->weight[(size_t)i * n_in + s];
    } else {
        int ho = conv_out(L->h_in, L->kh, L->stride, L->pad);
        int wo = conv_out(L->w_in, L->kw, L->stride, L->pad);
        int co = i / (ho * wo), oy = (i / wo) % ho, ox = i % wo;
        for (int s = 0; s < n_in; ++s) coef[s] = 0.0;
        for (int ci = 0; ci < L->c_in; ++ci)
            for (int ky = 0; ky < L->kh; ++ky)
                for (int kx = 0; kx < L->kw; ++kx) {
                    int iy = oy * L->stride - L->pad + ky;
                    int ix = ox * L->stride - L->pad + kx;
                    if (iy < 0 || iy >= L->h_in || ix < 0 || ix >= L->w_in) continue;
                    coef[((size_t)ci * L->h_in + iy) * L->w_in + ix] =
                        (double)L->weight[(((size_t)co * L->c_in + ci) * L->kh + ky) * L->kw + kx];
                }
        i = co;                                  /* one bias per output channel */
    }
    *d = (double)L->bias[i];
}

/* Replace every neuron t of affine layer L in the expression (coef over the
 * layer's outputs) by its polyhedral bound.  For an affine neuron L = U =
 * w.prev + b, so both branches of replace_* give coef[t]*(w_t.prev + b_t).   */
static void replace_through_affine(const oracle_layer_t *L, const double *coef,
                                   double *next, double *d)
{
    int n_in = layer_n_in(L), n_out = layer_n_out(L);
    for (int s = 0; s < n_in; ++s) next[s] = 0.0;
    if (L->kind == 0) {
        for (int t = 0; t < n_out; ++t) {
            double c = coef[t];
            if (c == 0.0) continue;
            const float *w = L->weight + (size_t)t * n_in;
            for (int s = 0; s < n_in; ++s) next[s] += c * (double)w[s];
            *d += c * (double)L->bias[t];
        }
    } else {
        int ho = conv_out(L->h_in, L->kh, L->stride, L->pad);
        int wo = conv_out(L->w_in, L->kw, L->stride, L->pad);
        for (int t = 0; t < n_out; ++t) {
            double c = coef[t];
            if (c == 0.0) continue;
            int co = t / (ho * wo), oy = (t / wo) % ho, ox = t % wo;
            for (int ci = 0; ci < L->c_in; ++ci)
                for (int ky = 0; ky < L->kh; ++ky)
                    for (int kx = 0; kx < L->kw; ++kx) {
                        int iy = oy * L->stride - L->pad + ky;
                        int ix = ox * L->stride - L->pad + kx;
                        if (iy < 0 || iy >= L->h_in || ix < 0 || ix >= L->w_in) continue;
                        next[((size_t)ci * L->h_in + iy) * L->w_in + ix] +=
                            c * (double)L->weight[(((size_t)co * L->c_in + ci) * L->kh + ky) * L->kw + kx];
                    }
            *d += c * (double)L->bias[co];
        }
    }
}

/* Replace every ReLU neuron t by its polyhedral bound over the affine neuron
 * below it: L_t = lamL[t]*z_t, U_t = lamU[t]*z_t + nuU[t].
 * upper == 0: replace_lower; upper == 1: replace_upper.                      */
static void replace_through_relu(int n, int upper, const double *lamL, const double *lamU,
                                 const double *nuU, double *coef, double *d)
{
    for (int t = 0; t < n; ++t) {
        double c = coef[t];
        int use_L = upper ? !(c >= 0.0) : (c >= 0.0);
        if (use_L) {
            coef[t] = c * lamL[t];
        } else {
            coef[t] = c * lamU[t];
            *d += c * nuU[t];
        }
    }
}

/* SkipPoly (Appendix C, SkipPoly listing): the shape of a ReLU neuron t on top of affine
 * layer Lj is expressed two layers back,
 *   L_t = relu_n(prev)       = (l + u >= 0) ? prev[L] : 0
 *   U_t = compute_upper(prev) = l >= 0 ? prev[U] : u <= 0 ? 0 : u/(u-l) * prev[U] - u*l/(u-l)
 * with prev[L] = prev[U] = w_t.a + b_t over the inputs a of the affine layer, so one traversal
 * round replaces the ReLU neurons by expressions over a directly:
 *   coefficient c  ->  c * (slope * w_t[s]) on every a_s,  constant += c * (slope * b_t + intercept).
 * row: scratch of n_in doubles.                                                              */
static void replace_through_relu_skip(const oracle_layer_t *Lj, int upper, const double *lamL,
                                      const double *lamU, const double *nuU, const double *coef,
                                      double *next, double *row, double *d)
{
    int n_in = layer_n_in(Lj), n_out = layer_n_out(Lj);
    for (int s = 0; s < n_in; ++s) next[s] = 0.0;
    for (int t = 0; t < n_out; ++t) {
        double c = coef[t];
        if (c == 0.0) continue;
        int use_L = upper ? !(c >= 0.0) : (c >= 0.0);
        double slope = use_L ? lamL[t] : lamU[t];
        double intercept = use_L ? 0.0 : nuU[t];
        double b;
        affine_row(Lj, t, row, &b);
        for (int s = 0; s < n_in; ++s) next[s] += c * (slope * row[s]);
        *d += c * (slope * b + intercept);
    }
}

/* simplify_lower / simplify_upper summed over the input neurons. */
static double concretize(int n, int upper, const double *coef, double d,
                         const double *l0, const double *u0)
{
    double acc = d;
    for (int s = 0; s < n; ++s) {
        double c = coef[s];
        if (c >= 0.0) acc += c * (upper ? u0[s] : l0[s]);
        else          acc += c * (upper ? l0[s] : u0[s]);
    }
    return acc;
}

/* The Relu transformer for one neuron with concrete bounds (l,u) of the
 * affine neuron below it. */
static void relu_relaxation(double l, double u, int decision_fp32, double *lamL, double *lamU,
                            double *nuU, unsigned char *code, double *margin)
{
    int active, inactive, pick_one;
    if (decision_fp32) {
        float lf = (float)l, uf = (float)u;
        volatile float sum = lf + uf;
        active = lf >= 0.0f;
        inactive = uf <= 0.0f;
        pick_one = sum >= 0.0f;
    } else {
        active = l >= 0.0;
        inactive = u <= 0.0;
        pick_one = (l + u) >= 0.0;
    }
    *lamL = pick_one ? 1.0 : 0.0;                        /* relu_n          */
    if (active)        { *lamU = 1.0; *nuU = 0.0; *code = 1; }   /* compute_upper */
    else if (inactive) { *lamU = 0.0; *nuU = 0.0; *code = 0; }
    else {
        *lamU = u / (u - l);
        *nuU = -(u * l) / (u - l);
        *code = (unsigned char)(2 + pick_one);
    }
    double m = fabs(l);
    if (fabs(u) < m) m = fabs(u);
    if (fabs(l + u) < m) m = fabs(l + u);
    double scale = fabs(l) > fabs(u) ? fabs(l) : fabs(u);
    *margin = m / (1.0 + scale);
}

/* One box: bounds of every affine neuron, layer after layer
 * (flow(forward, priority = layer)). */
static int one_box(const oracle_layer_t *layers, int n_layers, const float *center, float eps,
                   float clip_lo, float clip_hi, int decision_fp32, int max_backsteps_all,
                   const int *backsteps_per_layer, int skip_form, const int *skip_from,
                   double *lb, double *ub, unsigned char *codes, double *margins)
{
    int n0 = layer_n_in(&layers[0]);
    int n_max = n0, n_total = 0;
    for (int k = 0; k < n_layers; ++k) {
        int n = layer_n_out(&layers[k]);
        if (n > n_max) n_max = n;
        n_total += n;
    }
    double *l0 = malloc(sizeof(double) * n0), *u0 = malloc(sizeof(double) * n0);
    double *coef = malloc(sizeof(double) * n_max), *next = malloc(sizeof(double) * n_max);
    double *lamL = malloc(sizeof(double) * n_total), *lamU = malloc(sizeof(double) * n_total);
    double *nuU = malloc(sizeof(double) * n_total);
    double *row = malloc(sizeof(double) * n_max);
    int *off = malloc(sizeof(int) * (n_layers + 1));
    /* Residual connections: pend + off[t] holds coefficients over the outputs of layer t that
     * wait for the traversal to come down to that layer (has[t] != 0). */
    double *pend = calloc((size_t)n_total, sizeof(double));
    int *has = calloc((size_t)n_layers, sizeof(int));
    if (!l0 || !u0 || !coef || !next || !lamL || !lamU || !nuU || !off || !row || !pend || !has) return 1;

    /* The box endpoints are binary32 values: fl(c -/+ eps) clipped. */
    for (int s = 0; s < n0; ++s) {
        volatile float lo = center[s] - eps, hi = center[s] + eps;
        float lo_c = lo < clip_lo ? clip_lo : lo;
        float hi_c = hi > clip_hi ? clip_hi : hi;
        l0[s] = (double)lo_c;
        u0[s] = (double)hi_c;
    }
    off[0] = 0;
    for (int k = 0; k < n_layers; ++k) off[k + 1] = off[k] + layer_n_out(&layers[k]);

    int code_off = 0;
    for (int k = 0; k < n_layers; ++k) {
        int n_k = layer_n_out(&layers[k]);
        /* how many traversal steps the expressions of this layer take: all of them, or p */
        int max_backsteps = backsteps_per_layer ? backsteps_per_layer[k] : max_backsteps_all;
        for (int i = 0; i < n_k; ++i) {
            for (int upper = 0; upper < 2; ++upper) {
                double d;
                affine_row(&layers[k], i, coef, &d);
                /* A neuron of a layer with a residual connection is an affine neuron whose prev
                 * also holds neuron i of layer skip_from[k], with weight 1. */
                if (skip_from && skip_from[k] >= 0) {
                    pend[off[skip_from[k]] + i] += 1.0;
                    has[skip_from[k]] = 1;
                }
                int steps = 0;
                int j = k - 1;                 /* coef is over the outputs of layer j */
                for (; j >= 0; --j) {
                    if (max_backsteps >= 0 && steps >= max_backsteps) break;
                    if (has[j]) {
                        /* priority -layer: neurons of layer j are replaced only now, with all the
                         * coefficient they have gathered */
                        int n_j = layer_n_out(&layers[j]);
                        for (int t = 0; t < n_j; ++t) { coef[t] += pend[off[j] + t]; pend[off[j] + t] = 0.0; }
                        has[j] = 0;
                    }
                    if (skip_form && layers[j].relu_after) {
                        replace_through_relu_skip(&layers[j], upper, lamL + off[j], lamU + off[j],
                                                  nuU + off[j], coef, next, row, &d);
                    } else {
                        if (layers[j].relu_after)
                            replace_through_relu(layer_n_out(&layers[j]), upper, lamL + off[j],
                                                 lamU + off[j], nuU + off[j], coef, &d);
                        if (skip_from && skip_from[j] >= 0) {
                            /* coef is over the affine neurons of layer j = W_j a_{j-1} + b_j + a_s */
                            int sfrom = skip_from[j], n_j = layer_n_out(&layers[j]);
                            for (int t = 0; t < n_j; ++t) pend[off[sfrom] + t] += coef[t];
                            has[sfrom] = 1;
                        }
                        replace_through_affine(&layers[j], coef, next, &d);
                    }
                    double *tmp = coef; coef = next; next = tmp;
                    ++steps;
                }
                double v;
                if (j < 0) {
                    v = concretize(n0, upper, coef, d, l0, u0);
                } else {
                    /* Stopped early (DeepPoly_p, Section 6.2): simplify against the
                     * concrete bounds of the neurons reached: relu(l), relu(u) of
                     * layer j when a ReLU follows it, else its own l, u.  With residual
                     * connections the expression may also hold neurons of lower layers
                     * (coefficients that were still waiting): map(simplify_*) treats every
                     * neuron of the expression alike, each with its total coefficient. */
                    v = d;
                    for (int t2 = j; t2 >= 0; --t2) {
                        if (t2 < j && !has[t2]) continue;
                        int n_t = layer_n_out(&layers[t2]);
                        double *lt = next, *ut = malloc(sizeof(double) * n_t);
                        if (!ut) return 1;
                        for (int t = 0; t < n_t; ++t) {
                            double l = lb[off[t2] + t], u = ub[off[t2] + t];
                            if (layers[t2].relu_after) { l = l >= 0.0 ? l : 0.0; u = u >= 0.0 ? u : 0.0; }
                            lt[t] = l; ut[t] = u;
                        }
                        if (t2 == j) {
                            if (has[j]) {
                                for (int t = 0; t < n_t; ++t) { coef[t] += pend[off[j] + t]; pend[off[j] + t] = 0.0; }
                                has[j] = 0;
                            }
                            v += concretize(n_t, upper, coef, 0.0, lt, ut);
                        } else {
                            v += concretize(n_t, upper, pend + off[t2], 0.0, lt, ut);
                            for (int t = 0; t < n_t; ++t) pend[off[t2] + t] = 0.0;
                            has[t2] = 0;
                        }
                        free(ut);
                    }
                }
                if (upper) ub[off[k] + i] = v; else lb[off[k] + i] = v;
            }
        }
        if (layers[k].relu_after) {
            for (int t = 0; t < n_k; ++t) {
                unsigned char code; double margin;
                relu_relaxation(lb[off[k] + t], ub[off[k] + t], decision_fp32, &lamL[off[k] + t],
                                &lamU[off[k] + t], &nuU[off[k] + t], &code, &margin);
                if (codes) codes[code_off + t] = code;
                if (margins) margins[code_off + t] = margin;
            }
            code_off += n_k;
        }
    }
    free(l0); free(u0); free(coef); free(next); free(lamL); free(lamU); free(nuU); free(off); free(row);
    free(pend); free(has);
    return 0;
}

/* Number of affine neurons (sum over layers) and of ReLU neurons. */
int oracle_num_neurons(const oracle_layer_t *layers, int n_layers)
{
    int n = 0;
    for (int k = 0; k < n_layers; ++k) n += layer_n_out(&layers[k]);
    return n;
}

int oracle_num_relu_neurons(const oracle_layer_t *layers, int n_layers)
{
    int n = 0;
    for (int k = 0; k < n_layers; ++k)
        if (layers[k].relu_after) n += layer_n_out(&layers[k]);
    return n;
}

/*
 * lb, ub: [batch][n_total] float64, affine layers concatenated in order.
 * codes, margins (optional, may be NULL): [batch][n_relu].
 * max_backsteps < 0: full DeepPoly.  max_backsteps = p >= 0: DeepPoly_p
 * (Section 6.2: the traversal runs for p iterations at every affine layer; one
 * iteration here is one affine layer of the network together with the Relu
 * layer on top of it, so that p = number of affine layers is full DeepPoly).
 * backsteps_per_layer (optional, [n_layers]): a step count per affine layer,
 * overriding max_backsteps; this covers the other certifiers of Appendix C
 * that differ from DeepPoly only in where they traverse:
 *   IBP listing:       Affine -> map(simplify_*) of prev.dot(w)+b, no traversal: 0 everywhere;
 *   CROWN-IBP listing: the same, except curr[last_layer] == 1 -> backsubs_*: 0, ..., 0, -1,
 * with the Relu transformer (relu(l), relu(u), relu_n, compute_upper) unchanged.
 * skip_form != 0: the SkipPoly listing (ReLU shapes expressed two layers back; one traversal
 * round per ReLU layer).
 * (A traversal that stops early with such a connection still open simplifies the waiting coefficients
 * against the concrete bounds of their own layer, like every other neuron left in the expression.)
 * skip_from (optional, [n_layers]): residual connections.  skip_from[k] = s >= 0 (s <= k-2, equal widths)
 * makes layer k compute W_k a_{k-1} + b_k + a_s with a_s the outputs of layer s (after its ReLU, if it
 * has one); -1 = none.  Reading: such a neuron is the listing's Affine neuron whose prev holds neurons
 * of two layers (its own row of W_k over layer k-1, weight 1 on neuron i of layer s); the traversal's
 * priority -layer then replaces the neurons of the highest layer first, so the coefficient on a_s waits
 * until the rest of the expression has come down to layer s.
 * n_threads: boxes are independent and are the only parallel axis.
 * Returns 0, or 1 on allocation failure, 2 on a malformed network.
 */
int oracle_backsub(const oracle_layer_t *layers, int n_layers, const float *centers, float eps,
                   int batch, float clip_lo, float clip_hi, int decision_fp32, int max_backsteps,
                   const int *backsteps_per_layer, int skip_form, const int *skip_from,
                   int n_threads, double *lb, double *ub, unsigned char *codes, double *margins)
{
    if (n_layers < 1 || batch < 0) return 2;
    for (int k = 1; k < n_layers; ++k)
        if (layer_n_in(&layers[k]) != layer_n_out(&layers[k - 1])) return 2;
    if (skip_from) {
        /* residual connections: not in the SkipPoly form */
        if (skip_form) return 2;
        for (int k = 0; k < n_layers; ++k) {
            int sfrom = skip_from[k];
            if (sfrom < 0) continue;
            if (sfrom > k - 2 || layer_n_out(&layers[sfrom]) != layer_n_out(&layers[k])) return 2;
        }
    }
    int n0 = layer_n_in(&layers[0]);
    int n_total = oracle_num_neurons(layers, n_layers);
    int n_relu = oracle_num_relu_neurons(layers, n_layers);
    int err = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        int e = one_box(layers, n_layers, centers + (size_t)b * n0, eps, clip_lo, clip_hi,
                        decision_fp32, max_backsteps, backsteps_per_layer, skip_form, skip_from,
                        lb + (size_t)b * n_total,
                        ub + (size_t)b * n_total, codes ? codes + (size_t)b * n_relu : NULL,
                        margins ? margins + (size_t)b * n_relu : NULL);
        if (e) {
#pragma omp atomic write
            err = e;
        }
    }
    return err;
}

int oracle_deeppoly(const oracle_layer_t *layers, int n_layers, const float *centers, float eps,
                    int batch, float clip_lo, float clip_hi, int decision_fp32, int max_backsteps,
                    int n_threads, double *lb, double *ub, unsigned char *codes, double *margins)
{
    return oracle_backsub(layers, n_layers, centers, eps, batch, clip_lo, clip_hi, decision_fp32,
                          max_backsteps, NULL, 0, NULL, n_threads, lb, ub, codes, margins);
}

/*
 * ReuseCert (Appendix C, ReuseCert listing; Section 6.1): every neuron keeps polyhedral bounds
 * L, U expressed over the input layer (stop_traverse(n) = n[layer] <= 1), so an affine neuron's
 * traversal is a single round: each ReLU neuron below is replaced by its stored L / U.
 *   Affine, first layer:  L = U = prev.dot(w) + b (already over the input).
 *   Affine, later layers: L = backsubs_lower_L(prev.dot(w)+b): coefficient c of ReLU neuron t is
 *                         replaced by c*L_t if c >= 0 else c*U_t (upper: swapped); L_t, U_t are
 *                         affine expressions over the input.
 *   Relu:  l = prev[L].map(simplify_lower), u = prev[U].map(simplify_upper);
 *          L = relu_n(l,u,prev) = (l+u >= 0) ? prev[L] : 0
 *          U = compute_upper(l,u,prev) = l >= 0 ? prev[U] : u <= 0 ? 0 : u/(u-l)*prev[U] - u*l/(u-l).
 * The listing stores concrete bounds only for the first and the last affine layer; here the
 * l, u that the Relu transformer computes are reported for every affine layer (for the first and
 * last layer they are the listing's own backsubs_lower/upper values).
 * An affine layer directly on an affine layer uses the lower layer's L, U unchanged.
 */
static int reusecert_box(const oracle_layer_t *layers, int n_layers, const float *center, float eps,
                         float clip_lo, float clip_hi, int decision_fp32,
                         double *lb, double *ub, unsigned char *codes, double *margins)
{
    int n0 = layer_n_in(&layers[0]);
    int n_max = n0;
    for (int k = 0; k < n_layers; ++k) {
        int n = layer_n_out(&layers[k]);
        if (n > n_max) n_max = n;
    }
    size_t mat = (size_t)n_max * n0;
    double *l0 = malloc(sizeof(double) * n0), *u0 = malloc(sizeof(double) * n0);
    /* below: L, U (coefficients [neuron][input] and constants) of the outputs of the layer below */
    double *CLb = malloc(sizeof(double) * mat), *CUb = malloc(sizeof(double) * mat);
    double *dLb = malloc(sizeof(double) * n_max), *dUb = malloc(sizeof(double) * n_max);
    double *CL = malloc(sizeof(double) * mat), *CU = malloc(sizeof(double) * mat);
    double *dL = malloc(sizeof(double) * n_max), *dU = malloc(sizeof(double) * n_max);
    double *row = malloc(sizeof(double) * n_max);
    if (!l0 || !u0 || !CLb || !CUb || !dLb || !dUb || !CL || !CU || !dL || !dU || !row) return 1;
    for (int s = 0; s < n0; ++s) {
        volatile float lo = center[s] - eps, hi = center[s] + eps;
        float lo_c = lo < clip_lo ? clip_lo : lo;
        float hi_c = hi > clip_hi ? clip_hi : hi;
        l0[s] = (double)lo_c;
        u0[s] = (double)hi_c;
    }
    int off = 0, code_off = 0;
    for (int k = 0; k < n_layers; ++k) {
        int n_k = layer_n_out(&layers[k]);
        int n_prev = layer_n_in(&layers[k]);
        for (int i = 0; i < n_k; ++i) {
            double b;
            affine_row(&layers[k], i, row, &b);
            double *cl = CL + (size_t)i * n0, *cu = CU + (size_t)i * n0;
            if (k == 0) {
                for (int s = 0; s < n0; ++s) cl[s] = cu[s] = row[s];
                dL[i] = dU[i] = b;
            } else {
                for (int s = 0; s < n0; ++s) cl[s] = cu[s] = 0.0;
                double a_l = b, a_u = b;
                for (int t = 0; t < n_prev; ++t) {
                    double c = row[t];
                    if (c == 0.0) continue;
                    /* replace_lower: c >= 0 ? c*n[L] : c*n[U];  replace_upper: c >= 0 ? c*n[U] : c*n[L] */
                    const double *pl = (c >= 0.0 ? CLb : CUb) + (size_t)t * n0;
                    const double *pu = (c >= 0.0 ? CUb : CLb) + (size_t)t * n0;
                    for (int s = 0; s < n0; ++s) { cl[s] += c * pl[s]; cu[s] += c * pu[s]; }
                    a_l += c * (c >= 0.0 ? dLb[t] : dUb[t]);
                    a_u += c * (c >= 0.0 ? dUb[t] : dLb[t]);
                }
                dL[i] = a_l; dU[i] = a_u;
            }
            lb[off + i] = concretize(n0, 0, cl, dL[i], l0, u0);
            ub[off + i] = concretize(n0, 1, cu, dU[i], l0, u0);
        }
        /* shapes of this layer's outputs, over the input, for the layer above */
        for (int t = 0; t < n_k; ++t) {
            double lamL = 1.0, lamU = 1.0, nuU = 0.0;
            if (layers[k].relu_after) {
                unsigned char code; double margin;
                relu_relaxation(lb[off + t], ub[off + t], decision_fp32, &lamL, &lamU, &nuU, &code, &margin);
                if (codes) codes[code_off + t] = code;
                if (margins) margins[code_off + t] = margin;
            }
            const double *cl = CL + (size_t)t * n0, *cu = CU + (size_t)t * n0;
            double *bl = CLb + (size_t)t * n0, *bu = CUb + (size_t)t * n0;
            for (int s = 0; s < n0; ++s) { bl[s] = lamL * cl[s]; bu[s] = lamU * cu[s]; }
            dLb[t] = lamL * dL[t];
            dUb[t] = lamU * dU[t] + nuU;
        }
        if (layers[k].relu_after) code_off += n_k;
        off += n_k;
    }
    free(l0); free(u0); free(CLb); free(CUb); free(dLb); free(dUb); free(CL); free(CU); free(dL); free(dU);
    free(row);
    return 0;
}

/* Same outputs as oracle_deeppoly, for the ReuseCert certifier. */
int oracle_reusecert(const oracle_layer_t *layers, int n_layers, const float *centers, float eps,
                     int batch, float clip_lo, float clip_hi, int decision_fp32, int n_threads,
                     double *lb, double *ub, unsigned char *codes, double *margins)
{
    if (n_layers < 1 || batch < 0) return 2;
    for (int k = 1; k < n_layers; ++k)
        if (layer_n_in(&layers[k]) != layer_n_out(&layers[k - 1])) return 2;
    int n0 = layer_n_in(&layers[0]);
    int n_total = oracle_num_neurons(layers, n_layers);
    int n_relu = oracle_num_relu_neurons(layers, n_layers);
    int err = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        int e = reusecert_box(layers, n_layers, centers + (size_t)b * n0, eps, clip_lo, clip_hi,
                              decision_fp32, lb + (size_t)b * n_total, ub + (size_t)b * n_total,
                              codes ? codes + (size_t)b * n_relu : NULL,
                              margins ? margins + (size_t)b * n_relu : NULL);
        if (e) {
#pragma omp atomic write
            err = e;
        }
    }
    return err;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
