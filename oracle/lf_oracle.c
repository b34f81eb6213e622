/*
 * lf_oracle.c -- float64 CPU oracle for one pass of an L-layer, N-wide sigmoid MLP.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is the plain definition of what the
 * CUDA library must compute, written out slowly and obviously: no blocking, no fusion, no
 * reordering beyond what the equations state.  It shares no code, header, table or helper
 * with the CUDA path and neither includes the other.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may build or call it.
 *
 * What it follows (arXiv 1801.04928, "Leapfrogging for parallelism in deep neural networks"):
 *   Section 2, Eq. x   : a^0 = x                      (the paper's "layer 1" is the input)
 *   Section 2, Eq. z   : z^l = w^l a^{l-1} + b^l      (bias reading, see below)
 *   Section 2, Eq. a   : a^l = sigma(z^l)             (sigmoid by default; lfo_set_activation)
 *   Section 2, Eq. bp1 : delta^L = grad_a C (.) sigma'(z^L)
 *   Section 2, Eq. bp2 : delta^l = ((w^{l+1})^T delta^{l+1}) (.) sigma'(z^l)
 *   Section 2, Eq. bp3 : dC/db^l_j = delta^l_j
 *   Section 2, Eq. bp4 : dC/dw^l_jk = a^{l-1}_k delta^l_j
 *   Section 3, Algorithm 1 : the leapfrog schedule with k threads (lfo_backward_leapfrog)
 *   Section 1 ("k threads or k gpus") : one GPU's pass of the schedule on S GPUs (lfo_backward_shard)
 *   Section 2 (equations "generally valid") : the same pass for layers of different widths
 *                            (lfo_forward_widths, lfo_backward_widths)
 *   (not in the paper)     : the gradient-descent step that consumes Eq. bp4, w - eta dC/dw
 *                            (lfo_sgd_step); the paper ends with the gradients of one pass
 *
 * Readings taken where the paper is silent or garbled:
 *   - Eq. z prints no bias although b^l is defined and Eq. bp3 differentiates by it: the
 *     bias is added, z = w a + b.
 *   - Indexing: this code counts L WEIGHT layers l = 1..L with a^0 = x.  The paper numbers
 *     the input as layer 1, so paper layer p is l = p - 1 here and the paper's L is L + 1.
 *   - All layers, input and output included, are N wide (except in the *_widths functions).
 *   - C is the quadratic cost C = 1/2 sum_b ||a^L_b - y_b||^2 (a SUM over the B samples,
 *     no 1/B), hence grad_a C = a^L - y.  (The *_cross_entropy functions are the same pass
 *     under a second cost, see there.)
 *   - Mini-batch (B > 1) is an extension: every sample is an independent column; bp3 and
 *     bp4 are summed over the samples.
 *   - Algorithm 1 never applies bp3/bp4 at the top layer L; that is an omission.  The
 *     parent computes them there.
 *   - k >= L: the parent loop would run past the first weight layer; it stops at l = 1 and
 *     the threads find nothing to do.
 *
 * Storage (zero-based C arrays, everything contiguous, sample-major vectors):
 *   w[L][N][N]  w[l-1][j][k] = weight from neuron k of layer l-1 to neuron j of layer l
 *   b[L][N], x[B][N], y[B][N], z[L][B][N], a[L+1][B][N] (a[0] = x), delta[L][B][N],
 *   gw[L][N][N], gb[L][N].
 * Every array is double except w, whose element type is LFO_W_T: the file is compiled
 * twice, once with double (finite-difference pins need perturbations below fp32
 * resolution) and once with float (the fp32 weights of a large network are promoted
 * element by element instead of being copied to an 8-byte array first).
 *
 * Parity status of every function here: PINNED (central finite differences of lfo_cost,
 * closed forms, rank-1 / grad_b invariants, schedule invariance and coverage; see
 * tests/test_oracle_pins.py).
 */
#include <math.h>
#include <pthread.h>
#include <stdlib.h>
#include <string.h>

#ifndef LFO_W_T
#define LFO_W_T double
#endif
typedef LFO_W_T lfo_w_t;

#define IDX2(i, j, n) ((size_t)(i) * (size_t)(n) + (size_t)(j))

int lfo_weight_bytes(void) { return (int)sizeof(lfo_w_t); }

/* sigma(t) = 1 / (1 + e^{-t}), evaluated without overflow for either sign of t. */
static double lfo_sigmoid(double t)
{
    if (t >= 0.0) {
        return 1.0 / (1.0 + exp(-t));
    } else {
        double e = exp(t);
        return e / (1.0 + e);
    }
}

/* sigma'(t) = sigma(t) (1 - sigma(t)). */
static double lfo_sigmoid_prime(double t)
{
    double s = lfo_sigmoid(t);
    return s * (1.0 - s);
}

double lfo_sigma(double t) { return lfo_sigmoid(t); }
double lfo_sigma_prime(double t) { return lfo_sigmoid_prime(t); }

/* The activation function of Eq. a and its derivative in Eq. bp1 / bp2.  The paper writes sigma
 * for it and says its equations hold generally; the sigmoid is the default and what every
 * workload of the paper's kind uses.  Two more are offered so that an implementation's choice of
 * activation can be checked: tanh, and the rectifier max(t, 0) with derivative [t > 0] (taken as
 * 0 at t = 0).  The choice is a property of the whole pass, so it is a setting of this library
 * instance rather than an argument of every function. */
enum { LFO_ACT_SIGMOID = 0, LFO_ACT_TANH = 1, LFO_ACT_RELU = 2 };
static int lfo_activation = LFO_ACT_SIGMOID;

int lfo_set_activation(int kind)
{
    if (kind < LFO_ACT_SIGMOID || kind > LFO_ACT_RELU) return -1;
    lfo_activation = kind;
    return 0;
}

static double lfo_act(double t)
{
    if (lfo_activation == LFO_ACT_TANH) return tanh(t);
    if (lfo_activation == LFO_ACT_RELU) return t > 0.0 ? t : 0.0;
    return lfo_sigmoid(t);
}

static double lfo_act_prime(double t)
{
    if (lfo_activation == LFO_ACT_TANH) {
        double h = tanh(t);
        return 1.0 - h * h;
    }
    if (lfo_activation == LFO_ACT_RELU) return t > 0.0 ? 1.0 : 0.0;
    return lfo_sigmoid_prime(t);
}

/* Eq. x, Eq. z, Eq. a: the forward pass.  a has L+1 slabs of B*N, a[0] := x. */
void lfo_forward(int L, int N, int B, const lfo_w_t *w, const double *b, const double *x,
                 double *z, double *a)
{
    size_t slab = (size_t)B * (size_t)N;
    memcpy(a, x, slab * sizeof(double));                                  /* Eq. x */
    for (int l = 1; l <= L; ++l) {
        const lfo_w_t *wl = w + (size_t)(l - 1) * N * N;
        const double *bl = b + (size_t)(l - 1) * N;
        const double *aprev = a + (size_t)(l - 1) * slab;
        double *zl = z + (size_t)(l - 1) * slab;
        double *al = a + (size_t)l * slab;
        for (int s = 0; s < B; ++s) {
            for (int j = 0; j < N; ++j) {
                double acc = 0.0;
                for (int k = 0; k < N; ++k)
                    acc += (double)wl[IDX2(j, k, N)] * aprev[IDX2(s, k, N)];
                zl[IDX2(s, j, N)] = acc + bl[j];                          /* Eq. z */
                al[IDX2(s, j, N)] = lfo_act(zl[IDX2(s, j, N)]);           /* Eq. a */
            }
        }
    }
}

/* Quadratic cost C = 1/2 sum_b sum_j (a^L_bj - y_bj)^2 of an already computed forward pass. */
double lfo_cost(int L, int N, int B, const double *a, const double *y)
{
    const double *aL = a + (size_t)L * B * N;
    double c = 0.0;
    for (size_t i = 0; i < (size_t)B * N; ++i) {
        double d = aL[i] - y[i];
        c += d * d;
    }
    return 0.5 * c;
}

/* Eq. bp1 with grad_a C = a^L - y. */
void lfo_output_error(int N, int B, const double *aL, const double *y, const double *zL,
                      double *deltaL)
{
    for (size_t i = 0; i < (size_t)B * N; ++i)
        deltaL[i] = (aL[i] - y[i]) * lfo_act_prime(zL[i]);
}

/* Eq. bp2 at one layer: delta^l = ((w^{l+1})^T delta^{l+1}) (.) sigma'(z^l).
 * w_up is w^{l+1} (N x N, row-major), delta_up is delta^{l+1}, z_l is z^l. */
void lfo_delta_step(int N, int B, const lfo_w_t *w_up, const double *delta_up,
                    const double *z_l, double *delta_l)
{
    for (int s = 0; s < B; ++s) {
        for (int k = 0; k < N; ++k) {
            double acc = 0.0;
            for (int j = 0; j < N; ++j)                    /* ((w^{l+1})^T delta^{l+1})_k */
                acc += (double)w_up[IDX2(j, k, N)] * delta_up[IDX2(s, j, N)];
            delta_l[IDX2(s, k, N)] = acc * lfo_act_prime(z_l[IDX2(s, k, N)]);
        }
    }
}

/* Eq. bp3 summed over the samples: gb_j = sum_b delta_bj. */
void lfo_grad_b(int N, int B, const double *delta_l, double *gb_l)
{
    for (int j = 0; j < N; ++j) {
        double acc = 0.0;
        for (int s = 0; s < B; ++s)
            acc += delta_l[IDX2(s, j, N)];
        gb_l[j] = acc;
    }
}

/* Eq. bp4 summed over the samples: gw_jk = sum_b a^{l-1}_bk delta^l_bj. */
void lfo_grad_w(int N, int B, const double *delta_l, const double *a_prev, double *gw_l)
{
    for (int j = 0; j < N; ++j) {
        for (int k = 0; k < N; ++k) {
            double acc = 0.0;
            for (int s = 0; s < B; ++s)
                acc += a_prev[IDX2(s, k, N)] * delta_l[IDX2(s, j, N)];
            gw_l[IDX2(j, k, N)] = acc;
        }
    }
}

/* One entry of Eq. bp4 (for spot checks of matrices too large to materialise). */
double lfo_grad_w_entry(int N, int B, const double *delta_l, const double *a_prev, int j,
                        int k)
{
    double acc = 0.0;
    for (int s = 0; s < B; ++s)
        acc += a_prev[IDX2(s, k, N)] * delta_l[IDX2(s, j, N)];
    return acc;
}

/* bp3 and bp4 at layer l (1-based), results stored ("saved to shared memory" in
 * Algorithm 1) into gb / gw.  gw may be NULL: then only gb is produced. */
static void lfo_emit_layer(int l, int N, int B, const double *delta_l, const double *a,
                           double *gw, double *gb)
{
    size_t slab = (size_t)B * (size_t)N;
    lfo_grad_b(N, B, delta_l, gb + (size_t)(l - 1) * N);
    if (gw)
        lfo_grad_w(N, B, delta_l, a + (size_t)(l - 1) * slab, gw + (size_t)(l - 1) * N * N);
}

/* Everything below Eq. bp1: the caller has put delta^L into the top slab of `delta`; bp2
 * downwards, bp3/bp4 at every layer (L included). */
void lfo_backward_below_top(int L, int N, int B, const lfo_w_t *w, const double *z,
                            const double *a, double *delta, double *gw, double *gb)
{
    size_t slab = (size_t)B * (size_t)N;
    lfo_emit_layer(L, N, B, delta + (size_t)(L - 1) * slab, a, gw, gb);
    for (int l = L - 1; l >= 1; --l) {
        lfo_delta_step(N, B, w + (size_t)l * N * N, delta + (size_t)l * slab,
                       z + (size_t)(l - 1) * slab, delta + (size_t)(l - 1) * slab);
        lfo_emit_layer(l, N, B, delta + (size_t)(l - 1) * slab, a, gw, gb);
    }
}

/* Plain sequential backpropagation: bp1 at L, then bp2 downwards, bp3/bp4 everywhere. */
void lfo_backward_sequential(int L, int N, int B, const lfo_w_t *w, const double *z,
                             const double *a, const double *y, double *delta, double *gw,
                             double *gb)
{
    size_t slab = (size_t)B * (size_t)N;
    lfo_output_error(N, B, a + (size_t)L * slab, y, z + (size_t)(L - 1) * slab,
                     delta + (size_t)(L - 1) * slab);
    lfo_backward_below_top(L, N, B, w, z, a, delta, gw, gb);
}

/* ---- a second cost function: cross-entropy ------------------------------------------------
 * Section 2 leaves C open ("the cost function"; Eq. bp1 only needs grad_a C).  Besides the
 * quadratic cost this oracle knows the cross-entropy of sigmoid outputs,
 *     C = - sum_b sum_j [ y_bj ln a^L_bj + (1 - y_bj) ln(1 - a^L_bj) ]      (a sum, no 1/B),
 * whose gradient by the activations is grad_a C = (a - y) / (a (1 - a)).  Eq. bp1 is applied
 * as printed, grad_a C (.) sigma'(z^L); nothing is simplified here (that the product collapses
 * to a - y is what an implementation may use and what the tests then confirm). */
double lfo_cost_cross_entropy(int L, int N, int B, const double *a, const double *y)
{
    const double *aL = a + (size_t)L * B * N;
    double c = 0.0;
    for (size_t i = 0; i < (size_t)B * N; ++i)
        c -= y[i] * log(aL[i]) + (1.0 - y[i]) * log(1.0 - aL[i]);
    return c;
}

void lfo_output_error_cross_entropy(int N, int B, const double *aL, const double *y, const double *zL,
                                    double *deltaL)
{
    for (size_t i = 0; i < (size_t)B * N; ++i) {
        double grad_a = (aL[i] - y[i]) / (aL[i] * (1.0 - aL[i]));
        deltaL[i] = grad_a * lfo_act_prime(zL[i]);                     /* Eq. bp1 */
    }
}

void lfo_backward_sequential_cross_entropy(int L, int N, int B, const lfo_w_t *w, const double *z,
                                           const double *a, const double *y, double *delta,
                                           double *gw, double *gb)
{
    size_t slab = (size_t)B * (size_t)N;
    lfo_output_error_cross_entropy(N, B, a + (size_t)L * slab, y, z + (size_t)(L - 1) * slab,
                                   delta + (size_t)(L - 1) * slab);
    lfo_backward_below_top(L, N, B, w, z, a, delta, gw, gb);
}

/* ---- Algorithm 1: k threads, each recomputing the chain, each saving its own layers ----- */

typedef struct {
    int j, k, L, N, B;
    const lfo_w_t *w;
    const double *z, *a;
    const double *delta_start;  /* delta^{L-j}, computed by the parent               */
    double *delta, *gw, *gb;    /* shared result arrays                              */
    int *writer;                /* writer[l-1] = thread that saved layer l           */
    int *writes;                /* writes[l-1] = how many times layer l was saved    */
    long long bp2_steps;        /* how many bp2 applications this thread performed   */
} lfo_thread_arg;

/* The work of thread j of Algorithm 1, which starts from delta^{L-j} (computed by the parent).
 * Its layers are the residue class (L - l) mod k = j below its start: l = L-j-k, L-j-2k, ...
 * (Theorem 1: the k classes together cover every layer the parent did not do).  The algorithm
 * lets a thread take whole groups of k chain steps for as long as a group's first step lies above
 * layer k, i.e. n_groups = ceil((L - k - j) / k) groups (none if L - k - j <= 0), so its lowest
 * layer is L - j - n_groups * k >= 1.  The thread walks the delta chain on its own -- Eq. bp2 at
 * EVERY layer from its start down to that lowest layer, in private buffers -- and applies
 * Eq. bp3 / bp4 only where the layer is one of its own.  (With the paper's numbering, in which the
 * input is layer 1, its layer p is l = p - 1 here and its L is L + 1 here.)  That this walk visits
 * and saves exactly the layers the printed procedure does is checked, for every size up to
 * paper-L = 21, by an integer-only walk of that procedure in the tests. */
static void *lfo_thread_main(void *argp)
{
    lfo_thread_arg *t = (lfo_thread_arg *)argp;
    const int k = t->k, start = t->L - t->j;
    const int room = t->L - k - t->j;                          /* > 0: the thread has work */
    const int n_groups = room > 0 ? (room + k - 1) / k : 0;
    const int lowest = start - n_groups * k;
    size_t slab = (size_t)t->B * (size_t)t->N;
    double *cur = (double *)malloc(slab * sizeof(double));
    double *nxt = (double *)malloc(slab * sizeof(double));
    memcpy(cur, t->delta_start, slab * sizeof(double));
    for (int l = start - 1; l >= lowest && n_groups > 0; --l) {
        lfo_delta_step(t->N, t->B, t->w + (size_t)l * t->N * t->N, cur,
                       t->z + (size_t)(l - 1) * slab, nxt);               /* bp2: delta^l */
        t->bp2_steps += 1;
        double *tmp = cur; cur = nxt; nxt = tmp;
        if ((t->L - l) % k == t->j % k) {                                 /* one of this thread's layers */
            lfo_emit_layer(l, t->N, t->B, cur, t->a, t->gw, t->gb);       /* bp3, bp4 */
            memcpy(t->delta + (size_t)(l - 1) * slab, cur, slab * sizeof(double));
            t->writer[l - 1] = t->j;
            __atomic_fetch_add(&t->writes[l - 1], 1, __ATOMIC_RELAXED);
        }
    }
    free(cur);
    free(nxt);
    return NULL;
}

/* Procedure Backpropagation(k) of Algorithm 1 with k real threads.
 *   writer[L] (out, may be NULL): which thread saved each layer; -1 = the parent.
 *   writes[L] (out, may be NULL): how often each layer was saved (Theorem 1: exactly once).
 *   bp2_total (out, may be NULL): bp2 applications summed over parent and threads (the
 *                                 redundant chain walks the paper's cost model leaves out).
 *   run_threads != 0: pthreads run concurrently; 0: the same procedures run one after the
 *                     other on the calling thread (identical arithmetic).
 * Returns 0, or -1 for invalid sizes. */
int lfo_backward_leapfrog(int L, int N, int B, int k, const lfo_w_t *w, const double *z,
                          const double *a, const double *y, double *delta, double *gw,
                          double *gb, int *writer, int *writes, long long *bp2_total,
                          int run_threads)
{
    if (L < 1 || N < 1 || B < 1 || k < 1) return -1;
    if (k > L) k = L;
    size_t slab = (size_t)B * (size_t)N;
    int *wr = writer ? writer : (int *)malloc((size_t)L * sizeof(int));
    int *ws = writes ? writes : (int *)malloc((size_t)L * sizeof(int));
    for (int l = 0; l < L; ++l) { wr[l] = -2; ws[l] = 0; }
    long long parent_bp2 = 0;

    /* Parent: bp1 at L (and bp3/bp4 there, the omission noted in the header). */
    lfo_output_error(N, B, a + (size_t)L * slab, y, z + (size_t)(L - 1) * slab,
                     delta + (size_t)(L - 1) * slab);
    lfo_emit_layer(L, N, B, delta + (size_t)(L - 1) * slab, a, gw, gb);
    wr[L - 1] = -1; ws[L - 1] += 1;
    /* Parent: bp2, bp3, bp4 at the k-1 layers below L. */
    for (int l = L - 1; l >= L - k + 1 && l >= 1; --l) {
        lfo_delta_step(N, B, w + (size_t)l * N * N, delta + (size_t)l * slab,
                       z + (size_t)(l - 1) * slab, delta + (size_t)(l - 1) * slab);
        parent_bp2 += 1;
        lfo_emit_layer(l, N, B, delta + (size_t)(l - 1) * slab, a, gw, gb);
        wr[l - 1] = -1; ws[l - 1] += 1;
    }
    /* Construct k threads; thread j starts from delta^{L-j}. */
    lfo_thread_arg *args = (lfo_thread_arg *)calloc((size_t)k, sizeof(lfo_thread_arg));
    pthread_t *tids = (pthread_t *)calloc((size_t)k, sizeof(pthread_t));
    for (int j = 0; j < k; ++j) {
        lfo_thread_arg *t = &args[j];
        t->j = j; t->k = k; t->L = L; t->N = N; t->B = B;
        t->w = w; t->z = z; t->a = a;
        t->delta_start = delta + (size_t)(L - j - 1) * slab;
        t->delta = delta; t->gw = gw; t->gb = gb;
        t->writer = wr; t->writes = ws; t->bp2_steps = 0;
        if (run_threads)
            pthread_create(&tids[j], NULL, lfo_thread_main, t);
        else
            lfo_thread_main(t);
    }
    if (run_threads)
        for (int j = 0; j < k; ++j) pthread_join(tids[j], NULL);          /* join t_j */
    long long total = parent_bp2;
    for (int j = 0; j < k; ++j) total += args[j].bp2_steps;
    if (bp2_total) *bp2_total = total;
    free(args);
    free(tids);
    if (!writer) free(wr);
    if (!writes) free(ws);
    return 0;
}

/* One step of plain gradient descent on every weight matrix: w_new = w - eta * gw, with gw the
 * Eq. bp4 gradients of a pass.  The paper has no counterpart (it ends with the gradients of
 * one pass); this is the textbook definition of the step that consumes them, element by
 * element in float64, so that a fused "gradient + update" kernel has something to be checked
 * against.  Biases are left to the caller. */
void lfo_sgd_step(int L, int N, const lfo_w_t *w, const double *gw, double eta, double *w_new)
{
    const size_t n = (size_t)L * N * N;
    for (size_t i = 0; i < n; ++i) w_new[i] = (double)w[i] - eta * gw[i];
}

/* ---- layers of different widths ----------------------------------------------------------
 * Section 2 gives the hidden layers one width N "for simplicity" and notes that the equations
 * hold generally.  Here they are written out once more for widths n_0 .. n_L (n_0 the input,
 * n_L the output): w^l is n_l x n_{l-1}, every per-layer array is the concatenation of its
 * layers' blocks in layer order without padding,
 *     w, gw : block l = [n_l][n_{l-1}]      b, gb : block l = [n_l]
 *     z, delta : block l = [B][n_l]         a : block l = [B][n_l], l = 0..L, block 0 = x
 * Same equations, same order of operations as the functions above; only the index ranges of
 * the sums follow the layer.  cross_entropy != 0 selects the second cost in Eq. bp1. */
void lfo_forward_widths(int L, const int *n, int B, const lfo_w_t *w, const double *b,
                        const double *x, double *z, double *a)
{
    memcpy(a, x, (size_t)B * (size_t)n[0] * sizeof(double));             /* Eq. x */
    const lfo_w_t *wl = w;
    const double *bl = b, *aprev = a;
    double *zl = z;
    for (int l = 1; l <= L; ++l) {
        int rows = n[l], cols = n[l - 1];
        double *al = (double *)aprev + (size_t)B * cols;
        for (int s = 0; s < B; ++s) {
            for (int j = 0; j < rows; ++j) {
                double acc = 0.0;
                for (int k = 0; k < cols; ++k)
                    acc += (double)wl[IDX2(j, k, cols)] * aprev[IDX2(s, k, cols)];
                zl[IDX2(s, j, rows)] = acc + bl[j];                       /* Eq. z */
                al[IDX2(s, j, rows)] = lfo_act(zl[IDX2(s, j, rows)]);     /* Eq. a */
            }
        }
        wl += (size_t)rows * cols;
        bl += rows;
        zl += (size_t)B * rows;
        aprev = al;
    }
}

void lfo_backward_widths(int L, const int *n, int B, int cross_entropy, const lfo_w_t *w,
                         const double *z, const double *a, const double *y, double *delta,
                         double *gw, double *gb)
{
    /* where each layer's block starts (index l = 1..L; a also has l = 0) */
    size_t *ow = (size_t *)malloc(((size_t)L + 2) * sizeof(size_t));
    size_t *oh = (size_t *)malloc(((size_t)L + 2) * sizeof(size_t));
    size_t *oa = (size_t *)malloc(((size_t)L + 2) * sizeof(size_t));
    ow[1] = 0; oh[1] = 0; oa[0] = 0;
    for (int l = 1; l <= L; ++l) {
        ow[l + 1] = ow[l] + (size_t)n[l] * (size_t)n[l - 1];
        oh[l + 1] = oh[l] + (size_t)n[l];
        oa[l] = oa[l - 1] + (size_t)n[l - 1];
    }
    for (int l = L; l >= 1; --l) {
        int rows = n[l], cols = n[l - 1];
        double *dl = delta + (size_t)B * oh[l];
        const double *zl = z + (size_t)B * oh[l];
        if (l == L) {                                                     /* Eq. bp1 */
            const double *aL = a + (size_t)B * oa[L];
            for (size_t i = 0; i < (size_t)B * rows; ++i) {
                double grad_a = cross_entropy ? (aL[i] - y[i]) / (aL[i] * (1.0 - aL[i]))
                                              : aL[i] - y[i];
                dl[i] = grad_a * lfo_act_prime(zl[i]);
            }
        } else {                                                          /* Eq. bp2 */
            int up = n[l + 1];
            const lfo_w_t *wu = w + ow[l + 1];                            /* w^{l+1}: up x rows */
            const double *du = delta + (size_t)B * oh[l + 1];
            for (int s = 0; s < B; ++s) {
                for (int k = 0; k < rows; ++k) {
                    double acc = 0.0;
                    for (int j = 0; j < up; ++j)
                        acc += (double)wu[IDX2(j, k, rows)] * du[IDX2(s, j, up)];
                    dl[IDX2(s, k, rows)] = acc * lfo_act_prime(zl[IDX2(s, k, rows)]);
                }
            }
        }
        for (int j = 0; j < rows; ++j) {                                  /* Eq. bp3 */
            double acc = 0.0;
            for (int s = 0; s < B; ++s) acc += dl[IDX2(s, j, rows)];
            gb[oh[l] + j] = acc;
        }
        if (gw) {                                                         /* Eq. bp4 */
            const double *ap = a + (size_t)B * oa[l - 1];
            double *gl = gw + ow[l];
            for (int j = 0; j < rows; ++j) {
                for (int k = 0; k < cols; ++k) {
                    double acc = 0.0;
                    for (int s = 0; s < B; ++s)
                        acc += ap[IDX2(s, k, cols)] * dl[IDX2(s, j, rows)];
                    gl[IDX2(j, k, cols)] = acc;
                }
            }
        }
    }
    free(ow);
    free(oh);
    free(oa);
}

/* ---- the schedule on k GPUs instead of k threads -------------------------------------------
 * Section 1 offers the leapfrog schedule for "k threads or k gpus".  On S GPUs nothing is shared:
 * every GPU walks the whole delta chain (as every thread of Algorithm 1 does) and applies
 * Eq. bp3 / bp4 only at its own layers, those with (L - l) mod S = r for GPU r -- the residue
 * classes Algorithm 1 gives its threads (see the header on the three ways the paper names them).
 * This is GPU r's pass: delta is written completely; gb and gw only at the layers of shard r, the
 * other layers' slabs are left as they were; wrote[l-1] (may be NULL) is set to 1 at those layers
 * and to 0 elsewhere.  Returns 0, or -1 for invalid sizes. */
int lfo_backward_shard(int L, int N, int B, int S, int r, const lfo_w_t *w, const double *z,
                       const double *a, const double *y, double *delta, double *gw, double *gb,
                       int *wrote)
{
    if (L < 1 || N < 1 || B < 1 || S < 1 || r < 0 || r >= S) return -1;
    size_t slab = (size_t)B * (size_t)N;
    lfo_output_error(N, B, a + (size_t)L * slab, y, z + (size_t)(L - 1) * slab,
                     delta + (size_t)(L - 1) * slab);                          /* bp1 */
    for (int l = L; l >= 1; --l) {
        if (l < L)
            lfo_delta_step(N, B, w + (size_t)l * N * N, delta + (size_t)l * slab,
                           z + (size_t)(l - 1) * slab, delta + (size_t)(l - 1) * slab);   /* bp2 */
        int mine = (L - l) % S == r;
        if (mine) lfo_emit_layer(l, N, B, delta + (size_t)(l - 1) * slab, a, gw, gb);    /* bp3, bp4 */
        if (wrote) wrote[l - 1] = mine;
    }
    return 0;
}
