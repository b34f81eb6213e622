// Internal declarations shared by the translation units of libleapfrog (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "leapfrog.h"

// Bits of the device status word (0 = clean).
enum : unsigned {
    LF_DEV_TIMEOUT_FLAG = 1u,     // a wait on a ready flag ran out
    LF_DEV_TIMEOUT_BARRIER = 2u,  // a wait on a group barrier ran out
    LF_DEV_BAD_CONFIG = 4u        // a kernel was launched with a shape it does not support
};

struct lf_graph_key {
    const void *w, *z, *a, *y;
    void *delta, *gw, *gb;
    int variant, gw_math;
    int shard;      // shard rank * 65536 + shard count
    int sgd;        // 1: the graph writes w - eta * gw instead of gw
    float eta;
    int cost;       // enum lf_cost baked into the Eq. bp1 kernel
    int act;        // enum lf_activation baked into the kernels
    bool operator==(const lf_graph_key& o) const {
        return w == o.w && z == o.z && a == o.a && y == o.y && delta == o.delta &&
               gw == o.gw && gb == o.gb && variant == o.variant && gw_math == o.gw_math &&
               sgd == o.sgd && (!sgd || eta == o.eta) && cost == o.cost && act == o.act && shard == o.shard;
    }
};

// Fused weight update of the gradient writers: w_sub == nullptr -> store the gradient g itself,
// else store w_sub[...] - eta * g (w_sub is the weight matrix of the same layer).
struct lf_sgd {
    const float* w_sub;
    float eta;
};
#ifdef __CUDACC__
// Eq. a and the derivative used by Eq. bp1 / bp2, the latter from the stored activation a = sigma(z)
__device__ __forceinline__ float lf_act(float t, int kind)
{
    if (kind == LF_ACT_TANH) return tanhf(t);
    if (kind == LF_ACT_RELU) return fmaxf(t, 0.0f);
    return 1.0f / (1.0f + expf(-t));
}
__device__ __forceinline__ float lf_act_prime(float a, int kind)
{
    if (kind == LF_ACT_TANH) return 1.0f - a * a;
    if (kind == LF_ACT_RELU) return a > 0.0f ? 1.0f : 0.0f;
    return a * (1.0f - a);
}
// one rounding: fma(-eta, g, w)
__device__ __forceinline__ float4 lf_sgd_apply4(float eta, float4 w, float4 g)
{
    return make_float4(fmaf(-eta, g.x, w.x), fmaf(-eta, g.y, w.y), fmaf(-eta, g.z, w.z), fmaf(-eta, g.w, w.w));
}
#endif

struct lf_ctx {
    int L, N, B, k, keff;    // N: the common width, or the widest layer of a context with per-layer widths
    // per-layer widths n_0..n_L and where each layer's block starts inside the caller's arrays
    // (in floats; the per-sample arrays multiply by B).  Uniform contexts fill them with N.
    bool uniform;            // all widths equal: every kernel family applies
    // what a single-launch (persistent) pass covers: all L layers of a uniform context; the L - 2
    // layers 2..L-1 when only the hidden layers n_1..n_{L-1} share a width (the top and the bottom
    // layer then run as launches of their own); pk_N = 0 when there is no such run
    int pk_N, pk_L;
    int* width;              // [L+1]  n_l
    size_t* off_w;           // [L+1]  off_w[l-1]: start of w^l (n_l x n_{l-1}); off_w[L]: total
    size_t* off_h;           // [L+1]  off_h[l-1]: n_1 + ... + n_{l-1} (b, gb; z, delta times B)
    size_t* off_a;           // [L+2]  off_a[l]:   n_0 + ... + n_{l-1} (a times B)
    int device;
    int sm_count;
    int smem_optin;  // max dynamic shared memory per block
    cudaStream_t stream;

    // options
    int opt_variant;
    int opt_gw_math;
    long long wait_budget_us;
    int use_graph;
    int opt_delta_math;      // enum lf_delta_math
    int tc_pair_kernels;     // 1: the tensor-core contractions may use the two-SM (CTA pair) kernels
    int opt_cost;            // enum lf_cost
    int opt_act;             // enum lf_activation
    int sgd_on;              // the current backward call is lf_backward_sgd
    float sgd_eta;
    const float* sgd_w;      // its weights (what the update is subtracted from)
    int shard_rank, shard_count;  // layer l is this context's iff (L - l) % shard_count == shard_rank
    int withhold;            // test hook: one chain CTA withholds its published delta values

    // workspace (device)
    float* partial;          // partial column sums of the delta matvec: [row_chunks][N]
    unsigned* counters;      // arrival counters, one per column strip (self-resetting)
    unsigned* sync_words;    // persistent kernels: ready flags + barrier words (zeroed per call)
    size_t sync_words_count;
    unsigned* status_dev;    // device status word
    unsigned* status_host;   // pinned mirror
    float* dg_partial;       // B > 1: K-split partial sums of the tensor-core delta GEMM
    float* sb_partial;       // 1 < B <= 16: row-chunk partial sums of the small-batch Eq. bp2 kernel

    // leapfrog workers as streams
    cudaStream_t* wstreams;  // keff streams
    cudaEvent_t* ready_ev;   // L events: delta^l is complete
    cudaEvent_t* done_ev;    // keff events: worker finished its layers
    cudaEvent_t fork_ev;

    // captured graph of the STREAMS variant
    cudaGraphExec_t graph_exec;
    lf_graph_key graph_key;
    bool graph_valid;
    int graph_launches;      // kernels inside the captured graph

    // persistent kernels: TMA descriptor of w (opaque 128-byte CUtensorMap) and the call epoch
    alignas(64) unsigned char w_map_storage[128];
    bool w_map_valid;
    const void* w_map_ptr;
    int w_map_wc;
    unsigned epoch;
    // the whole-columns fused kernel keeps a descriptor of its own (another box shape)
    alignas(64) unsigned char ck_map_storage[128];
    bool ck_map_valid;
    const void* ck_map_ptr;
    int ck_map_wc;
    int opt_fused_tiling;    // enum lf_fused_tiling
    // its form for layers of different widths: device copy of one tensor map per layer and the layer table
    void* ckw_dev;
    const void* ckw_ptr;     // the weights they describe
#if defined(LF_PK_TRACE) || defined(LF_CK_TRACE)
    unsigned long long* trace_dev;  // debug builds: per-step SM-clock stamps of two CTAs
#endif

    // host-buffer entry point staging
    float* stage;            // one allocation holding w, a, y, delta, gw, gb
    size_t stage_bytes;
    cudaStream_t h2d_stream; // host -> device copies of the host entry point
    cudaStream_t d2h_stream; // device -> host copies of its results, all on this one stream
    cudaEvent_t* w_ready_ev; // L events: w^l has arrived in staging
    cudaEvent_t* gw_done_ev; // L events: gw^l (and gb^l) are written
    cudaEvent_t small_ev, h2d_done_ev, d2h_done_ev;
    bool host_path_ready;    // the copy streams and events above all exist

    // LF_OPT_TIME_CALLS: two timing events around the last backward call
    int time_calls;
    cudaEvent_t t_begin_ev, t_end_ev;
    bool timed_call_pending;

    int last_cuda_error;
    lf_stats stats;
};

// Layer-sharded form: does this context do Eq. bp3/bp4 of layer l, and on which of its workers?
inline bool lf_layer_owned(const lf_ctx* c, int l) { return (c->L - l) % c->shard_count == c->shard_rank; }
inline int lf_layer_worker(const lf_ctx* c, int l) { return ((c->L - l) / c->shard_count) % c->keff; }

#define LF_CUDA_TRY(ctx, expr)                                  \
    do {                                                        \
        cudaError_t e__ = (expr);                               \
        if (e__ != cudaSuccess) {                               \
            (ctx)->last_cuda_error = (int)e__;                  \
            return LF_ECUDA;                                    \
        }                                                       \
    } while (0)

// ---- launchers (each enqueues on `s` and returns the cudaError_t of the launch) -------------

// B = 1 kernels
// A layer's matrix is n_out x n_in, row-major: n_out neurons above, n_in below.
cudaError_t lfk_forward_matvec(const float* w_l, const float* b_l, const float* a_prev,
                               float* z_l, float* a_l, int n_out, int n_in, int act, cudaStream_t s);
cudaError_t lfk_copy_input(const float* x, float* a0, size_t n, cudaStream_t s);
cudaError_t lfk_output_error(const float* aL, const float* y, float* deltaL, float* gbL, int N,
                             int B, int cost, int act, cudaStream_t s);
int lfk_delta_row_chunks(int n_up);  // number of row chunks the delta matvec splits n_up rows into
cudaError_t lfk_delta_matvec(const float* w_up, const float* delta_up, const float* a_l,
                             float* delta_l, float* gb_l, float* partial, unsigned* counters,
                             int n_up, int n_l, int act, cudaStream_t s);
cudaError_t lfk_gw_rank1(const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                         lf_sgd sgd, cudaStream_t s);

// B > 1 kernels (fp32 on the CUDA cores)
cudaError_t lfk_forward_gemm(const float* w_l, const float* b_l, const float* a_prev,
                             float* z_l, float* a_l, int n_out, int n_in, int B, int act, cudaStream_t s);
cudaError_t lfk_delta_gemm(const float* w_up, const float* delta_up, const float* a_l,
                           float* delta_l, int n_up, int n_l, int B, int act, cudaStream_t s);
cudaError_t lfk_gw_gemm_fp32(const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                             int B, lf_sgd sgd, cudaStream_t s);
cudaError_t lfk_grad_b_colsum(const float* delta_l, float* gb_l, int N, int B, cudaStream_t s);
// Eq. bp2 for a handful of samples (B <= lfk_small_batch_max()): w read once at the memory rate, fp32
int lfk_small_batch_max();
size_t lfk_delta_small_batch_scratch_floats(int n_up, int n_l, int B);
cudaError_t lfk_delta_small_batch(const float* w_up, const float* delta_up, const float* a_l, float* delta_l,
                                  float* partial, unsigned* counters, int n_up, int n_l, int B, int act, cudaStream_t s);

// ---- persistent single-launch backward (B = 1) ---------------------------------------------
size_t lf_sync_words_needed(const lf_ctx* c);           // unsigned words of flag/barrier workspace
bool lf_persistent_supported(const lf_ctx* c, int variant);
int lf_auto_variant(const lf_ctx* c);                   // table lookup for LF_VARIANT_AUTO
int lf_backward_persistent(lf_ctx* c, int variant, const float* w, const float* a, const float* y, float* delta,
                           float* gw, float* gb, const float* w_sub, int top_given, int depth_shift);
void lf_persistent_release(lf_ctx* c);
int lf_fused_tiling(const lf_ctx* c);                   // which fused kernel a context gets (enum lf_fused_tiling)
constexpr int LF_COLUMNS_AUTO_MAX_N = 640;    // widths up to which LF_VARIANT_AUTO takes the fused pass with whole columns
constexpr int LF_COLUMNS_FUSED_MAX_N = 768;   // widths up to which a fused pass takes whole columns (LF_FUSED_TILING_AUTO)
// the fused pass with whole columns per CTA (one hop through L2 per layer, no clusters)
bool lf_columns_supported(const lf_ctx* c);
int lf_backward_columns(lf_ctx* c, const float* w, const float* a, const float* y, float* delta, float* gw,
                        float* gb, const float* w_sub, int top_given, int depth_shift);
// ... and over all layers of a context whose layers differ in width (one sample)
bool lf_columns_widths_supported(const lf_ctx* c);
int lf_backward_columns_widths(lf_ctx* c, const float* w, const float* a, const float* y, float* delta, float* gw,
                               float* gb, const float* w_sub);
void lf_columns_release(lf_ctx* c);

// ---- TF32 tensor-core weight-gradient contraction (B > 1) ------------------------------------
bool lf_tf32_supported(const lf_ctx* c);
int lf_gw_gemm_tf32(lf_ctx* c, const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                    lf_sgd sgd, cudaStream_t s, int* launches);
void lf_tf32_release(lf_ctx* c);

// ---- 3xTF32 tensor-core delta recurrence (B > 1) ----------------------------------------------
size_t lf_delta_tc_scratch_bytes(const lf_ctx* c);
bool lf_delta_tc_supported(const lf_ctx* c);
int lf_delta_gemm_tc(lf_ctx* c, const float* w_up, const float* delta_up, const float* a_l, float* delta_l,
                     int n_up, int n_l, int math, cudaStream_t s, int* launches);
int lf_forward_gemm_tc(lf_ctx* c, const float* w_l, const float* b_l, const float* a_prev, float* z_l, float* a_l,
                       int n_out, int n_in, int math, cudaStream_t s, int* launches);
