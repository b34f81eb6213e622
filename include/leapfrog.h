/*
 * leapfrog.h -- C ABI of the sm_100a library for one pass of an L-layer, N-wide sigmoid
 * multi-layer perceptron with the weight-gradient work interleaved over k workers
 * ("leapfrogging", arXiv 1801.04928).
 *
 * Indexing.  The library counts L WEIGHT layers l = 1..L with a^0 = x.  The paper numbers
 * the input as its layer 1, so paper layer p is l = p - 1 here.  C arrays are zero-based:
 * slab l-1 of an array holds the quantity of layer l.
 *
 * Layouts.  All tensors are float32, contiguous, 16-byte aligned and live in DEVICE memory
 * owned by the caller (except for the *_host entry point, which says so).  With B samples:
 *     w     [L][N][N]   w[l-1][j][k] = weight from neuron k of layer l-1 to neuron j of layer l
 *     b     [L][N]
 *     x, y  [B][N]      sample-major; B = 1 is the paper's vector form
 *     z     [L][B][N]
 *     a     [L+1][B][N] a[0] = x
 *     delta [L][B][N]
 *     gw    [L][N][N]   same indexing as w
 *     gb    [L][N]
 * N must be a multiple of 4 (128-bit accesses); other sizes are rejected with LF_EINVAL.
 * (lf_create_widths gives every layer its own width; its layouts are stated there.)
 *
 * Execution.  Calls enqueue work on the context's stream and return; lf_sync() waits for it
 * and reports device-side status.  The library never allocates or frees tensors; a context
 * owns only its workspace (flags, reduction scratch, helper streams and events).  Nothing
 * here throws or aborts; every entry point returns LF_OK (0) or a negative code.  There is
 * no CPU fallback: without a CUDA device every compute entry point fails with LF_ECUDA.
 * A context is not thread-safe; use one per host thread.
 */
#ifndef LEAPFROG_H
#define LEAPFROG_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lf_ctx lf_ctx;

enum lf_status {
    LF_OK = 0,
    LF_EINVAL = -1,    /* L, N, B or k < 1, N not a multiple of 4, unknown option or value  */
    LF_ENULL = -2,     /* a required pointer is NULL                                         */
    LF_EALIGN = -3,    /* a tensor pointer is not 16-byte aligned                            */
    LF_ERESOURCE = -4, /* the device cannot hold the requested configuration co-resident     */
    LF_ECUDA = -5,     /* a CUDA call failed; lf_last_cuda_error() gives the cudaError_t     */
    LF_ETIMEOUT = -6,  /* a bounded device-side wait ran out; outputs are undefined          */
    LF_ENOMEM = -7,    /* workspace allocation failed                                        */
    LF_ECAPACITY = -8  /* size is beyond the fixed capacity of an allocation-free entry point */
};

/* How lf_backward schedules Eq. bp4 (the weight gradients) against the delta chain.  The two
 * persistent variants exist for B = 1 and N <= 16384; elsewhere, and when the device cannot
 * keep the grid co-resident, lf_backward uses LF_VARIANT_STREAMS instead -- lf_get_stats()
 * reports the variant that actually ran. */
enum lf_variant {
    LF_VARIANT_AUTO = 0,       /* pick from the built-in per-(N,B) table of measurements      */
    LF_VARIANT_STREAMS = 1,    /* one launch per layer; the k leapfrog workers are k streams  */
    LF_VARIANT_PERSISTENT = 2, /* one persistent launch; the k workers are k CTA groups       */
    LF_VARIANT_FUSED = 3       /* one persistent launch; the pass that reads a tile of
                                  w^{l+1} for Eq. bp2 also stores the same tile of gw^{l+1}   */
};

/* Arithmetic of the B > 1 weight-gradient contraction. */
enum lf_gw_math {
    LF_GW_MATH_AUTO = 0, /* TF32 tensor cores when B > 16 and the shape is supported; up to 16
                            samples Eq. bp4 is a store stream and stays fp32 (faster and exact)  */
    LF_GW_MATH_FP32 = 1, /* fp32 FMA on the CUDA cores                                        */
    LF_GW_MATH_TF32 = 2  /* inputs rounded to TF32, fp32 accumulation in tensor memory        */
};

/* Arithmetic of the B > 1 delta recurrence and forward pass (Eq. bp2 and Eq. z as N x N x B
 * contractions). */
enum lf_delta_math {
    LF_DELTA_MATH_AUTO = 0,  /* tensor cores when B > 1 and the device supports it; Eq. bp2 for 2 to
                                8 samples, and for 9 to 16 samples of layers at least 2048 wide,
                                stays fp32 on the CUDA cores (a batched matrix-vector product
                                that reads w^{l+1} once, at the memory rate)                      */
    LF_DELTA_MATH_FP32 = 1,  /* fp32 FMA on the CUDA cores                                        */
    LF_DELTA_MATH_3XTF32 = 2, /* tensor cores; every operand split into two TF32 numbers, three
                                products per term, fp32 accumulation: fp32-level accuracy        */
    LF_DELTA_MATH_TF32_BF16 = 3 /* tensor cores; the product of the two high parts in TF32, the two
                                cross terms (each below 2^-11 of the product) in BF16: eight
                                instead of twelve instructions per K stage, about 2^-20 per
                                term.  Applies to CTA-pair tiles (one-CTA tiles keep three TF32
                                products).  Never chosen by AUTO: as measured, splitting the
                                operands, not the tensor cores, then bounds the kernel.          */
};

/* Tiling of the tensor-core contractions (B > 1): one CTA per tile, or a pair of CTAs (two
 * multiprocessors) per tile, which share one operand and halve the traffic per multiply-add. */
enum lf_tc_tiling {
    LF_TC_TILING_AUTO = 0,   /* CTA pairs where they apply and the device can co-schedule them  */
    LF_TC_TILING_ONE_SM = 1, /* one CTA per tile                                                */
    LF_TC_TILING_TWO_SM = 2  /* CTA pairs: Eq. bp4 at every B (up to 256 samples the delta operand
                                of a row block stays in shared memory, beyond that both operands
                                stream), Eq. bp2 / Eq. z for B > 128 and N >= 512; other sizes use
                                ONE_SM                                                          */
};

/* Tiling of the fused single-launch pass (LF_VARIANT_FUSED, B = 1). */
enum lf_fused_tiling {
    LF_FUSED_TILING_AUTO = 0,     /* whole columns at the widths where the delta hand-off is the bound */
    LF_FUSED_TILING_CLUSTERS = 1, /* thread-block clusters own column strips, their CTAs row blocks of
                                     them; partial sums cross the cluster's shared memory             */
    LF_FUSED_TILING_COLUMNS = 2   /* every CTA owns whole columns (all rows): delta crosses CTAs once
                                     per layer, and each CTA stores the rows of gw it finished itself
                                     (in lf_backward_sgd it reads those rows of w from memory once
                                     more, where CLUSTERS takes them from the tile the chain holds)   */
};

/* The cost function C of Eq. bp1, delta^L = grad_a C (.) sigma'(z^L); Section 2 leaves it open
 * ("the cost function").  Both are sums over the B samples (no 1/B). */
enum lf_cost {
    LF_COST_QUADRATIC = 0,     /* C = 1/2 sum ||a^L - y||^2: delta^L = (a^L - y) (.) sigma'(z^L)  */
    LF_COST_CROSS_ENTROPY = 1  /* C = -sum [y ln a^L + (1-y) ln(1-a^L)] on the sigmoid outputs:
                                  grad_a C = (a^L - y) / (a^L (1 - a^L)), so delta^L = a^L - y   */
};

/* The activation function sigma of Eq. a (and sigma' of Eq. bp1 / bp2, taken from the stored
 * activations).  The paper writes a general sigma; the sigmoid is the default. */
enum lf_activation {
    LF_ACT_SIGMOID = 0, /* sigma(t) = 1 / (1 + e^{-t}),  sigma' = a (1 - a)                        */
    LF_ACT_TANH = 1,    /* sigma(t) = tanh t,             sigma' = 1 - a^2                         */
    LF_ACT_RELU = 2     /* sigma(t) = max(t, 0),          sigma' = [a > 0]  (0 where t <= 0)       */
};

/*
 * LF_OPT_SHARD_COUNT = S > 1 and LF_OPT_SHARD_RANK = r (in the enum below) select the
 * layer-sharded form.  The paper offers its schedule for "k threads or k gpus": with S GPUs every GPU holds w, z, a, runs the whole delta
 * chain for itself, and does Eq. bp4 (and, for B > 1, Eq. bp3) only for the layers it owns,
 *     layer l belongs to shard (L - l) mod S,
 * so that nothing is exchanged during the pass and the gradients end up distributed by owner.
 * A context with S > 1 writes delta completely (and gb for B = 1, where it is delta), and gw^l
 * (gb^l for B > 1; w_new^l in lf_backward_sgd) only for its own layers; the other layers' blocks
 * of those arrays are not touched.  Inside the shard the k leapfrog workers share the shard's
 * layers in turn: worker ((L - l) / S) mod k.  The S contexts are independent: one per GPU, or
 * several on one GPU writing into one gw array, give together exactly what one unsharded
 * context writes.  Every variant takes a sharded context (the fused pass skips the stores of
 * other shards' tiles).
 */
enum lf_option {
    LF_OPT_VARIANT = 1,       /* enum lf_variant                                              */
    LF_OPT_GW_MATH = 2,       /* enum lf_gw_math                                              */
    LF_OPT_WAIT_BUDGET_US = 3,/* upper bound of any device-side wait, microseconds (>= 1)     */
    LF_OPT_USE_GRAPH = 4,     /* 0/1: replay the STREAMS variant from a captured CUDA graph   */
    LF_OPT_DELTA_MATH = 6,    /* enum lf_delta_math                                           */
    LF_OPT_TC_TILING = 7,     /* enum lf_tc_tiling                                            */
    LF_OPT_COST = 8,          /* enum lf_cost (default LF_COST_QUADRATIC)                     */
    LF_OPT_ACTIVATION = 9,    /* enum lf_activation (default LF_ACT_SIGMOID); applies to
                                 lf_forward and lf_backward alike, so set it before both.
                                 LF_COST_CROSS_ENTROPY needs the sigmoid: lf_backward returns
                                 LF_EINVAL for any other pairing                              */
    LF_OPT_SHARD_COUNT = 10,  /* S >= 1 (default 1): the paper's "k gpus" form (Section 1), see
                                 above; setting it puts the rank back to 0                    */
    LF_OPT_SHARD_RANK = 11,   /* r, 0 <= r < S: which of the S shards this context is         */
    LF_OPT_FUSED_TILING = 12, /* enum lf_fused_tiling                                         */
    LF_OPT_TIME_CALLS = 13,   /* 0/1 (default 0): bracket every backward call with two events on
                                 the context's stream; lf_sync then puts the elapsed device time
                                 of the last one into lf_stats.last_backward_ms                 */
    LF_OPT_WITHHOLD = 5       /* test hook, 0 (off), 1 or 2.  1, single-launch variants: one CTA does
                                 not publish its share of delta.  2, tensor-core weight-gradient
                                 kernels (B > 1): one producer arms a stage and never loads it.
                                 Either way the bounded waits of the others expire and lf_sync()
                                 reports LF_ETIMEOUT (no fault, no hang)                          */
};

typedef struct lf_stats {
    int L, N, B, k;           /* sizes the context was created with                           */
    int k_effective;          /* min(k, L)                                                    */
    int variant;              /* variant the last lf_backward used (enum lf_variant)          */
    int gw_math;              /* arithmetic the last lf_backward used for Eq. bp4             */
    int sm_count;             /* multiprocessors of the device                                */
    int chain_ctas;           /* persistent variants: CTAs on the delta chain                 */
    int worker_ctas;          /* persistent variants: CTAs per leapfrog worker group          */
    int launches_forward;     /* kernels launched by the last lf_forward                      */
    int launches_backward;    /* kernels launched by the last lf_backward                     */
    unsigned int device_status; /* status word read by the last lf_sync (0 = clean)           */
    long long workspace_bytes;  /* device memory owned by the context                         */
    int delta_math;           /* arithmetic the last lf_backward used for Eq. bp2 (B > 1)     */
    int gw_tiling;            /* tiling of the last TF32 weight-gradient launch (enum lf_tc_tiling,
                                 ONE_SM or TWO_SM; 0 if none ran)                             */
    int delta_tiling;         /* the same for the last tensor-core Eq. bp2 / Eq. z launch     */
    int cost;                 /* cost function the last lf_backward used (enum lf_cost)       */
    int activation;           /* activation the last lf_forward / lf_backward used            */
    int shard_rank;           /* LF_OPT_SHARD_RANK and LF_OPT_SHARD_COUNT of the last lf_backward */
    int shard_count;
    int fused_tiling;         /* tiling of the last fused single-launch pass (enum lf_fused_tiling,
                                 CLUSTERS or COLUMNS; 0 if the last pass was not a fused one)     */
    float last_backward_ms;   /* device time of the last lf_backward / lf_backward_sgd /
                                 lf_backward_host between two events on the context's stream, as
                                 of the last lf_sync (0 before the first; filled only while
                                 LF_OPT_TIME_CALLS is on)                                         */
} lf_stats;

/*
 * Create a context for networks of L weight layers, width N, B samples and k leapfrog
 * workers (Section 3: "k threads"; here CTA groups or streams).  k > L is legal and acts as
 * k = L.  Binds to the current CUDA device and allocates the workspace there.
 * *out receives the context; on failure *out is NULL.
 * Two options take their initial value from the environment, if set, so that a run can be steered
 * without touching the caller: LF_VARIANT = auto | streams | persistent | fused (LF_OPT_VARIANT) and
 * LF_FUSED_TILING = auto | clusters | columns (LF_OPT_FUSED_TILING), by name or by number; a later
 * lf_set_option overrides them, an unknown value is ignored.
 * Errors: LF_ENULL (out), LF_EINVAL (sizes), LF_ECUDA (no device / CUDA failure), LF_ENOMEM.
 */
int lf_create(lf_ctx** out, int L, int N, int B, int k);

/*
 * The same for a network whose layers differ in width (Section 2 gives only the hidden layers
 * a common width N and says the equations hold generally): widths is a HOST array of L + 1
 * ints, widths[0] = n_0 the width of the input x, widths[l] = n_l the number of neurons of
 * weight layer l, widths[L] = n_L the width of the output and of y.  Every width must be
 * >= 1 and a multiple of 4.  The array is copied; the caller may free it on return.
 *
 * Layouts: each array is the concatenation of its per-layer blocks, in layer order, with no
 * padding (all block starts stay 16-byte aligned because the widths are multiples of 4):
 *     w, gw    block l = [n_l][n_{l-1}] row-major, l = 1..L   (w^l_jk: neuron k below -> neuron j)
 *     b, gb    block l = [n_l]
 *     z, delta block l = [B][n_l]
 *     a        block l = [B][n_l], l = 0..L, a block 0 = x
 *     x [B][n_0],  y [B][n_L]
 * With all widths equal this is lf_create(L, widths[0], B, k) exactly, layouts included.
 * Otherwise, for one sample (B = 1), LF_VARIANT_FUSED -- and LF_VARIANT_AUTO, which picks it --
 * runs the whole pass as ONE launch whatever the widths are (the whole-columns tiling gives every
 * layer its own split of columns over the CTAs; up to 64 layers, widths up to 16384);
 * LF_VARIANT_STREAMS runs one launch per layer and step with the k workers as streams; and
 * LF_VARIANT_PERSISTENT, or LF_VARIANT_FUSED with LF_FUSED_TILING_CLUSTERS -- kernels written for
 * one common width -- run over the hidden layers n_1 .. n_{L-1} if those share a width (the
 * network of Section 2, whose input and output widths are left open; L >= 3), between per-layer
 * launches for the top and the bottom layer, and fall back to LF_VARIANT_STREAMS if they do not.
 * A mini-batch (B > 1) runs one launch per layer.  lf_get_stats() reports what ran, with N = the
 * widest layer.
 * The arithmetic options apply as for lf_create (B > 1: tensor-core contractions by default).  lf_forward, lf_backward,
 * lf_backward_sgd and lf_backward_host take such a context; lf_grad_w, which names no layer,
 * returns LF_EINVAL for it.
 * Errors: LF_ENULL (out, widths), LF_EINVAL (sizes), LF_ECUDA, LF_ENOMEM.
 */
int lf_create_widths(lf_ctx** out, int L, const int* widths, int B, int k);

/*
 * Use `cuda_stream` (a cudaStream_t, borrowed, must outlive the work enqueued on it) for
 * all subsequent calls.  NULL selects the legacy default stream (the initial setting).
 */
int lf_set_stream(lf_ctx* ctx, void* cuda_stream);

/* Set an option (enum lf_option).  LF_EINVAL for unknown keys or out-of-range values. */
int lf_set_option(lf_ctx* ctx, int key, long long value);

/*
 * Forward pass, Section 2 Eq. x, z, a:  a^0 = x;  z^l = w^l a^{l-1} + b^l;  a^l = sigma(z^l),
 * sigma(t) = 1 / (1 + e^{-t}).  (The printed Eq. z shows no bias; b^l is added, as Eq. bp3
 * presupposes.)  Reads w, b, x; writes all L slabs of z and all L+1 slabs of a (a[0] := x).
 */
int lf_forward(lf_ctx* ctx, const float* w, const float* b, const float* x, float* z,
               float* a);

/*
 * Backward pass under the quadratic cost C = 1/2 sum_b ||a^L_b - y_b||^2 (or, with
 * LF_OPT_COST = LF_COST_CROSS_ENTROPY, the cross-entropy cost, for which Eq. bp1 reads
 * delta^L = a^L - y):
 *   Eq. bp1  delta^L = (a^L - y) (.) sigma'(z^L)
 *   Eq. bp2  delta^l = ((w^{l+1})^T delta^{l+1}) (.) sigma'(z^l),  l = L-1 .. 1
 *   Eq. bp3  gb^l = sum_b delta^l_b
 *   Eq. bp4  gw^l = sum_b delta^l_b (a^{l-1}_b)^T
 * with Eq. bp3/bp4 of layer l done by leapfrog worker (L - l) mod k (Section 3, Algorithm 1;
 * the delta chain itself is computed once, not once per worker).  The top layer L, which
 * Algorithm 1 leaves out, is included.  z and a must be what lf_forward produced for the
 * same w (sigma' may be taken from a as a (1 - a)).  Reads w (layers 2..L), z, a, y; writes
 * every element of delta, gw and gb.  For B > 1 with TF32 math the inputs of Eq. bp4 are
 * rounded to TF32 and accumulated in fp32; everything else is fp32.
 */
int lf_backward(lf_ctx* ctx, const float* w, const float* z, const float* a, const float* y,
                float* delta, float* gw, float* gb);

/*
 * Eq. bp4 alone, for one layer:  gw_l = sum_b delta_l[b] (a_prev[b])^T  with delta_l = delta^l and
 * a_prev = a^{l-1}, both [B][N]; gw_l receives all N x N entries.  The same kernel, arithmetic
 * (LF_OPT_GW_MATH) and tiling as inside lf_backward, enqueued on the context's stream; the
 * result is bitwise what lf_backward writes into that layer's slab of gw.  Device pointers,
 * 16-byte aligned, owned by the caller.
 */
int lf_grad_w(lf_ctx* ctx, const float* delta_l, const float* a_prev, float* gw_l);

/*
 * Backward pass fused with one step of gradient descent on the weights.  (The paper has no
 * counterpart: it ends with the gradients of one pass.  This is the step that follows, folded
 * into the gradient writer so that gw is never stored and read back.)  As lf_backward, except
 * that in place of gw^l the call writes
 *     w_new^l = w^l - eta * gw^l,        l = 1..L,   w_new laid out like w ([L][N][N]),
 * every element of it, gw^l being the Eq. bp4 gradient of this pass (fp32, or TF32 products
 * for B > 1 under LF_GW_MATH_TF32).  Each element is one fused multiply-add of the fp32
 * gradient, fma(-eta, gw, w), i.e. one rounding.  w is only read; w_new must not overlap w
 * (the delta chain still reads w^{l+1} after w_new^{l+1} has been written).  delta and gb are
 * written as by lf_backward; the bias update b - eta * gb is left to the caller (N values per
 * layer).
 * Errors: as lf_backward; LF_EINVAL if eta is not finite or w_new overlaps w.
 */
int lf_backward_sgd(lf_ctx* ctx, const float* w, const float* z, const float* a, const float* y,
                    float eta, float* delta, float* w_new, float* gb);

/*
 * The same backward pass on HOST buffers (pageable or pinned; same layouts): w (layers 2..L, the
 * ones the pass reads), a, y are copied to device staging owned by the context (allocated on first use, counted in
 * workspace_bytes), delta, gw, gb are copied back.  z is not copied and not read (sigma' is taken
 * from a); it must still be non-NULL.  The copies are pipelined with the per-layer
 * schedule (LF_VARIANT_STREAMS): weights arrive top layer first on a copy stream, layer l is
 * processed as soon as w^{l+1} is there, and gw^l is sent back as soon as its worker has
 * written it, so both PCIe directions are busy at once (use pinned memory for that).  All work
 * is joined back into the context's stream.  The host buffers must stay valid until
 * lf_sync() returns.
 */
int lf_backward_host(lf_ctx* ctx, const float* w, const float* z, const float* a,
                     const float* y, float* delta, float* gw, float* gb);

/*
 * Wait for everything enqueued on the context's stream and read the device status word.
 * Returns LF_ETIMEOUT if a bounded device-side wait expired, LF_ECUDA on a CUDA error.
 */
int lf_sync(lf_ctx* ctx);

/* Worker that performs Eq. bp3/bp4 of layer l (1-based): (L - l) mod min(k, L); -1 if out of range.
 * In a sharded context: ((L - l) / S) mod min(k, L) for the shard's own layers, -1 for the others. */
int lf_owner(const lf_ctx* ctx, int l);

/* Copy the context's counters into *out. */
int lf_get_stats(lf_ctx* ctx, lf_stats* out);

/* cudaError_t of the last failed CUDA call of this context (0 if none). */
int lf_last_cuda_error(const lf_ctx* ctx);

/*
 * One delta-chain step (Eq. bp2, single sample) for callers that cannot allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for the library's users.)
 *
 *     delta_l[k] = (sum_j w_up[j][k] * delta_up[j]) * a_l[k] * (1 - a_l[k]),   k = 0..N-1
 *
 * w_up is w^{l+1} [N][N] row-major, delta_up is delta^{l+1} [N], a_l is a^l = sigma(z^l) [N],
 * delta_l receives delta^l [N]; all are device pointers, float32, 16-byte aligned, owned by
 * the caller.  The result is the same as the delta slab lf_backward writes for that layer.
 *
 * Who needs it: a process that has handed all of the GPU's memory to its own pool (an
 * inference server or a framework allocator that reserves HBM up front), where a cudaMalloc
 * made behind its back fails or fragments the pool; and a latency-critical loop that cannot
 * afford the device-wide synchronisation an allocation or a free implies.  Every other entry
 * point needs an lf_ctx, and lf_create allocates.  This one takes no context and calls no
 * allocating routine: the scratch its kernel needs (partial column sums and arrival counters)
 * is a fixed array inside the library image, about 1 MiB, resident on every GPU that loads the
 * library until the process exits.
 *
 * Limits and rules:
 *  - N must be a multiple of 4 and at most 4096; a larger N is LF_ECAPACITY (nothing is run).
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and remembers it; make that first call outside any stream capture.  With CUDA's
 *    default lazy loading that look-up is also the moment the driver loads this part of the
 *    library onto the device, which reserves the array and the kernel code there and synchronises
 *    the device: so make one warm-up call per device early -- BEFORE the process hands the
 *    remaining memory to its pool, and outside any latency-critical section.  If the device has no
 *    memory left for that, the call returns LF_ENOMEM and nothing is run.  Calls after the first
 *    one neither allocate nor synchronise.
 *  - All calls on a device share the one array.  Calls whose kernels may overlap on the GPU
 *    (different streams without an ordering between them, or several host threads) race on it
 *    and give wrong results; keep calls on one stream or order them with events.
 *  - `cuda_stream` is a cudaStream_t of the current device (NULL = legacy default stream).  The
 *    call enqueues a small memset of the counters and one kernel, and returns without waiting.
 * Errors: LF_ENULL, LF_EALIGN, LF_EINVAL (N), LF_ECAPACITY, LF_ERESOURCE (device ordinal
 * >= 64), LF_ENOMEM (first call on a device that cannot hold the array), LF_ECUDA.
 */
int lf_delta_step_static(const float* w_up, const float* delta_up, const float* a_l,
                         float* delta_l, int N, void* cuda_stream);

/* Static English text for a status code. */
const char* lf_strerror(int status);

/* Library version, major * 100 + minor. */
int lf_version(void);

/* Synchronise the stream, free the workspace and the context.  NULL is LF_ENULL. */
int lf_destroy(lf_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LEAPFROG_H */
