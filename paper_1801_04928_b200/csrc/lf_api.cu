// C ABI of libleapfrog: context, validation, scheduling of the per-layer kernels.
#include <new>
#include <stdlib.h>
#include <string.h>

#include "lf_internal.h"

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Initial value of an option from the environment: one of `names` (its index) or a number in range;
// anything else, or no variable, gives `fallback`.
int option_from_env(const char* var, const char* const* names, int count, int fallback)
{
    const char* e = getenv(var);
    if (!e || !*e) return fallback;
    for (int i = 0; i < count; ++i)
        if (strcmp(e, names[i]) == 0) return i;
    char* end = nullptr;
    const long v = strtol(e, &end, 10);
    return (end && *end == 0 && v >= 0 && v < count) ? (int)v : fallback;
}

int check_ptrs(const void* const* ps, int n)
{
    for (int i = 0; i < n; ++i)
        if (!ps[i]) return LF_ENULL;
    for (int i = 0; i < n; ++i)
        if (!aligned16(ps[i])) return LF_EALIGN;
    return LF_OK;
}

// Where layer l's block starts inside the caller's arrays (floats).
inline size_t w_at(const lf_ctx* c, int l) { return c->off_w[l - 1]; }                      // w, gw: l = 1..L
inline size_t v_at(const lf_ctx* c, int l) { return c->off_h[l - 1]; }                      // b, gb
inline size_t h_at(const lf_ctx* c, int l) { return (size_t)c->B * c->off_h[l - 1]; }       // z, delta
inline size_t a_at(const lf_ctx* c, int l) { return (size_t)c->B * c->off_a[l]; }           // a: l = 0..L

// LF_VARIANT_AUTO for layers of different widths (one sample): the single launch wherever it exists --
// measured against one launch per layer it is ahead at every shape tried (no launch gaps, the chain
// never leaves the SMs).
bool lf_widths_auto_single_launch(const lf_ctx*) { return true; }

// The persistent kernels are written for one common width (every cluster owns the same column strip
// of every layer): they serve uniform contexts and, for one sample, the run of hidden layers of a
// context whose input and output widths alone differ; other contexts run one launch per layer.
int resolve_variant(const lf_ctx* c)
{
    // layers of different widths, one sample: the fused pass with whole columns per CTA takes any
    // shape in one launch (where it was asked for; LF_VARIANT_AUTO: see below)
    if (!c->uniform && c->B == 1 && c->opt_fused_tiling != LF_FUSED_TILING_CLUSTERS &&
        (c->opt_variant == LF_VARIANT_FUSED || (c->opt_variant == LF_VARIANT_AUTO && lf_widths_auto_single_launch(c))) &&
        lf_columns_widths_supported(c))
        return LF_VARIANT_FUSED;
    if (!c->uniform && (c->B != 1 || c->pk_N <= 0)) return LF_VARIANT_STREAMS;
    return c->opt_variant != LF_VARIANT_AUTO ? c->opt_variant : lf_auto_variant(c);
}

int resolve_gw_math(const lf_ctx* c)
{
    if (c->B == 1) return LF_GW_MATH_FP32;  // rank-1: one multiply per element, nothing to contract
    if (c->opt_gw_math == LF_GW_MATH_FP32) return LF_GW_MATH_FP32;
    // up to 16 samples Eq. bp4 is a store stream (4B multiply-adds per 16 bytes): the fp32 writer is ahead
    // of the tensor-core tiles at every width measured (256 .. 8192), and exact
    if (c->opt_gw_math == LF_GW_MATH_AUTO && c->B <= 16) return LF_GW_MATH_FP32;
    return lf_tf32_supported(c) ? LF_GW_MATH_TF32 : LF_GW_MATH_FP32;
}

// Eq. bp4 (and, for a mini-batch, Eq. bp3) of layer l on stream s.
int enqueue_gradients(lf_ctx* c, int l, const float* a, const float* delta, float* gw, float* gb,
                      int gw_math, cudaStream_t s, int* launches)
{
    const float* d_l = delta + h_at(c, l);
    const float* a_prev = a + a_at(c, l - 1);
    float* gw_l = gw + w_at(c, l);
    const int n_out = c->width[l], n_in = c->width[l - 1];
    lf_sgd sgd = {nullptr, 0.f};
    if (c->sgd_on) { sgd.w_sub = c->sgd_w + w_at(c, l); sgd.eta = c->sgd_eta; }
    if (c->B == 1) {
        LF_CUDA_TRY(c, lfk_gw_rank1(d_l, a_prev, gw_l, n_out, n_in, sgd, s));
        *launches += 1;
    } else {
        if (gw_math == LF_GW_MATH_TF32) {
            int rc = lf_gw_gemm_tf32(c, d_l, a_prev, gw_l, n_out, n_in, sgd, s, launches);
            if (rc != LF_OK) return rc;
        } else {
            LF_CUDA_TRY(c, lfk_gw_gemm_fp32(d_l, a_prev, gw_l, n_out, n_in, c->B, sgd, s));
            *launches += 1;
        }
        LF_CUDA_TRY(c, lfk_grad_b_colsum(d_l, gb + v_at(c, l), n_out, c->B, s));
        *launches += 1;
    }
    return LF_OK;
}

// Arithmetic of the forward pass for B > 1 (Eq. z as a contraction).
int resolve_forward_math(const lf_ctx* c)
{
    if (c->B == 1 || c->opt_delta_math == LF_DELTA_MATH_FP32) return LF_DELTA_MATH_FP32;
    if (!lf_delta_tc_supported(c)) return LF_DELTA_MATH_FP32;
    return c->opt_delta_math == LF_DELTA_MATH_TF32_BF16 ? LF_DELTA_MATH_TF32_BF16 : LF_DELTA_MATH_3XTF32;
}

// Arithmetic of Eq. bp2 for B > 1.  A handful of samples is a batched matrix-vector product: fp32 on
// the CUDA cores at the memory rate beats tensor-core tiles that are nearly empty (unless the
// tensor cores are asked for by name).  Measured, whole pass per layer, widths 256 .. 8192: up to 8
// samples the fp32 kernel is ahead at every width; with 9 to 16 samples from a width of 2048.
int resolve_delta_math(const lf_ctx* c)
{
    if (c->B == 1 || c->opt_delta_math == LF_DELTA_MATH_FP32) return LF_DELTA_MATH_FP32;
    if (c->opt_delta_math == LF_DELTA_MATH_AUTO && c->sb_partial && c->B <= lfk_small_batch_max() &&
        (c->B <= 8 || c->N >= 2048))
        return LF_DELTA_MATH_FP32;
    if (!lf_delta_tc_supported(c)) return LF_DELTA_MATH_FP32;
    return c->opt_delta_math == LF_DELTA_MATH_TF32_BF16 ? LF_DELTA_MATH_TF32_BF16 : LF_DELTA_MATH_3XTF32;
}

// One delta-chain step on stream s: Eq. bp1 for l = L, Eq. bp2 below.
int enqueue_chain_step(lf_ctx* c, int l, const float* w, const float* a, const float* y,
                       float* delta, float* gb, cudaStream_t s, int* launches)
{
    const int L = c->L, B = c->B, n_l = c->width[l];
    float* d_l = delta + h_at(c, l);
    const float* a_l = a + a_at(c, l);
    float* gb_l = gb + v_at(c, l);
    if (l == L) {
        LF_CUDA_TRY(c, lfk_output_error(a_l, y, d_l, gb_l, n_l, B, c->opt_cost, c->opt_act, s));
    } else {
        const float* w_up = w + w_at(c, l + 1);  // w^{l+1}: n_{l+1} x n_l
        const float* d_up = delta + h_at(c, l + 1);
        const int n_up = c->width[l + 1];
        if (B == 1)
            LF_CUDA_TRY(c, lfk_delta_matvec(w_up, d_up, a_l, d_l, gb_l, c->partial, c->counters, n_up, n_l,
                                            c->opt_act, s));
        else if (c->stats.delta_math >= LF_DELTA_MATH_3XTF32) {
            int rc = lf_delta_gemm_tc(c, w_up, d_up, a_l, d_l, n_up, n_l, c->stats.delta_math, s, launches);
            if (rc != LF_OK) return rc;
            return LF_OK;
        } else if (B <= lfk_small_batch_max() && c->sb_partial)
            LF_CUDA_TRY(c, lfk_delta_small_batch(w_up, d_up, a_l, d_l, c->sb_partial, c->counters, n_up, n_l, B,
                                                 c->opt_act, s));
        else
            LF_CUDA_TRY(c, lfk_delta_gemm(w_up, d_up, a_l, d_l, n_up, n_l, B, c->opt_act, s));
    }
    *launches += 1;
    return LF_OK;
}

// The leapfrog schedule with streams: the chain runs on the context's stream and signals
// ready[l]; worker (L - l) mod k waits for it on its own stream and does Eq. bp3/bp4 there.
int enqueue_backward_streams(lf_ctx* c, const float* w, const float* a, const float* y,
                             float* delta, float* gw, float* gb, int gw_math, int* launches)
{
    cudaStream_t s = c->stream;
    LF_CUDA_TRY(c, cudaEventRecord(c->fork_ev, s));
    for (int j = 0; j < c->keff; ++j)
        LF_CUDA_TRY(c, cudaStreamWaitEvent(c->wstreams[j], c->fork_ev, 0));
    for (int l = c->L; l >= 1; --l) {
        int rc = enqueue_chain_step(c, l, w, a, y, delta, gb, s, launches);
        if (rc != LF_OK) return rc;
        if (!lf_layer_owned(c, l)) continue;      // another shard's layer
        LF_CUDA_TRY(c, cudaEventRecord(c->ready_ev[l - 1], s));
        int j = lf_layer_worker(c, l);
        LF_CUDA_TRY(c, cudaStreamWaitEvent(c->wstreams[j], c->ready_ev[l - 1], 0));
        rc = enqueue_gradients(c, l, a, delta, gw, gb, gw_math, c->wstreams[j], launches);
        if (rc != LF_OK) return rc;
    }
    for (int j = 0; j < c->keff; ++j) {
        LF_CUDA_TRY(c, cudaEventRecord(c->done_ev[j], c->wstreams[j]));
        LF_CUDA_TRY(c, cudaStreamWaitEvent(s, c->done_ev[j], 0));
    }
    return LF_OK;
}

void drop_graph(lf_ctx* c)
{
    if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
    c->graph_exec = nullptr;
    c->graph_valid = false;
}

int backward_streams(lf_ctx* c, const float* w, const float* z, const float* a, const float* y,
                     float* delta, float* gw, float* gb, int gw_math)
{
    int launches = 0;
    const bool graph_ok = c->use_graph && c->stream != nullptr &&
                          c->stream != cudaStreamLegacy && c->stream != cudaStreamPerThread;
    if (!graph_ok) {
        int rc = enqueue_backward_streams(c, w, a, y, delta, gw, gb, gw_math, &launches);
        c->stats.launches_backward = launches;
        return rc;
    }
    lf_graph_key key{w, z, a, y, delta, gw, gb, LF_VARIANT_STREAMS, gw_math * 16 + c->stats.delta_math,
                     c->shard_rank * 65536 + c->shard_count, c->sgd_on, c->sgd_eta, c->opt_cost, c->opt_act};
    if (!(c->graph_valid && c->graph_key == key)) {
        drop_graph(c);
        LF_CUDA_TRY(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
        int rc = enqueue_backward_streams(c, w, a, y, delta, gw, gb, gw_math, &launches);
        cudaGraph_t g = nullptr;
        cudaError_t e = cudaStreamEndCapture(c->stream, &g);
        if (rc != LF_OK) {
            if (g) cudaGraphDestroy(g);
            return rc;
        }
        if (e != cudaSuccess) {
            c->last_cuda_error = (int)e;
            return LF_ECUDA;
        }
        e = cudaGraphInstantiate(&c->graph_exec, g, 0);
        cudaGraphDestroy(g);
        if (e != cudaSuccess) {
            c->last_cuda_error = (int)e;
            c->graph_exec = nullptr;
            return LF_ECUDA;
        }
        c->graph_key = key;
        c->graph_valid = true;
        c->graph_launches = launches;
    }
    LF_CUDA_TRY(c, cudaGraphLaunch(c->graph_exec, c->stream));
    c->stats.launches_backward = c->graph_launches;
    return LF_OK;
}

// One sample, hidden layers n_1 = ... = n_{L-1} of one width, input and/or output of another (the
// network of the paper's Section 2): the top layer L and the bottom layer 1, whose matrices are not
// square, run as launches of their own around ONE persistent launch over layers 2..L-1.
//   stream:  Eq. bp1 (delta^L) -> Eq. bp2 with w^L (delta^{L-1}) -> persistent launch, which takes
//            delta^{L-1} as given and goes down to delta^2 -> Eq. bp2 with w^2 (delta^1)
//   workers: gw^L after delta^L and gw^1 after delta^1, on their leapfrog workers' streams
int backward_hidden_run(lf_ctx* c, int variant, const float* w, const float* a, const float* y, float* delta,
                        float* gw, float* gb, int gw_math)
{
    const int L = c->L;
    cudaStream_t s = c->stream;
    int launches = 0;
    LF_CUDA_TRY(c, cudaEventRecord(c->fork_ev, s));
    for (int j = 0; j < c->keff; ++j) LF_CUDA_TRY(c, cudaStreamWaitEvent(c->wstreams[j], c->fork_ev, 0));
    bool used[2] = {false, false};
    int worker[2] = {0, 0};
    const int ends[2] = {L, 1};
    for (int e = 0; e < 2; ++e) {
        const int l = ends[e];
        int rc;
        if (e == 0) {
            rc = enqueue_chain_step(c, L, w, a, y, delta, gb, s, &launches);            // delta^L
        } else {
            rc = enqueue_chain_step(c, 1, w, a, y, delta, gb, s, &launches);            // delta^1 from delta^2
        }
        if (rc != LF_OK) return rc;
        if (lf_layer_owned(c, l)) {
            LF_CUDA_TRY(c, cudaEventRecord(c->ready_ev[l - 1], s));
            worker[e] = lf_layer_worker(c, l);
            used[e] = true;
            LF_CUDA_TRY(c, cudaStreamWaitEvent(c->wstreams[worker[e]], c->ready_ev[l - 1], 0));
            rc = enqueue_gradients(c, l, a, delta, gw, gb, gw_math, c->wstreams[worker[e]], &launches);
            if (rc != LF_OK) return rc;
        }
        if (e == 0) {
            rc = enqueue_chain_step(c, L - 1, w, a, y, delta, gb, s, &launches);        // delta^{L-1}
            if (rc != LF_OK) return rc;
            rc = lf_backward_persistent(c, variant, w + w_at(c, 2), a + a_at(c, 1), y, delta + h_at(c, 2),
                                        gw + w_at(c, 2), gb + v_at(c, 2),
                                        c->sgd_on ? c->sgd_w + w_at(c, 2) : nullptr, 1, 1);
            if (rc != LF_OK) return rc;
            launches += 1;
        }
    }
    for (int e = 0; e < 2; ++e) {
        if (!used[e]) continue;
        LF_CUDA_TRY(c, cudaEventRecord(c->done_ev[worker[e]], c->wstreams[worker[e]]));
        LF_CUDA_TRY(c, cudaStreamWaitEvent(s, c->done_ev[worker[e]], 0));
    }
    c->stats.launches_backward = launches;
    return LF_OK;
}

}  // namespace

extern "C" {

int lf_version(void) { return 100; }

const char* lf_strerror(int status)
{
    switch (status) {
        case LF_OK: return "ok";
        case LF_EINVAL: return "invalid argument (sizes must be >= 1, N a multiple of 4, option in range)";
        case LF_ENULL: return "required pointer is NULL";
        case LF_EALIGN: return "tensor pointer is not 16-byte aligned";
        case LF_ERESOURCE: return "configuration cannot be made co-resident on this device";
        case LF_ECUDA: return "CUDA call failed (see lf_last_cuda_error)";
        case LF_ETIMEOUT: return "a bounded device-side wait expired; outputs are undefined";
        case LF_ENOMEM: return "workspace allocation failed";
        case LF_ECAPACITY: return "size exceeds the fixed capacity of this allocation-free entry point";
        default: return "unknown status";
    }
}

int lf_create(lf_ctx** out, int L, int N, int B, int k)
{
    if (!out) return LF_ENULL;
    *out = nullptr;
    if (L < 1 || N < 1 || B < 1 || k < 1 || (N & 3) != 0) return LF_EINVAL;
    int* widths = new (std::nothrow) int[(size_t)L + 1];
    if (!widths) return LF_ENOMEM;
    for (int l = 0; l <= L; ++l) widths[l] = N;
    const int rc = lf_create_widths(out, L, widths, B, k);
    delete[] widths;
    return rc;
}

int lf_create_widths(lf_ctx** out, int L, const int* widths, int B, int k)
{
    if (!out) return LF_ENULL;
    *out = nullptr;
    if (!widths) return LF_ENULL;
    if (L < 1 || B < 1 || k < 1) return LF_EINVAL;
    int N = 0;            // the widest layer
    bool uniform = true;
    for (int l = 0; l <= L; ++l) {
        if (widths[l] < 1 || (widths[l] & 3) != 0) return LF_EINVAL;
        if (widths[l] > N) N = widths[l];
        if (widths[l] != widths[0]) uniform = false;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LF_ECUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return LF_ECUDA;

    lf_ctx* c = new (std::nothrow) lf_ctx;
    if (!c) return LF_ENOMEM;
    memset(c, 0, sizeof(*c));
    c->L = L; c->N = N; c->B = B; c->k = k; c->keff = k < L ? k : L;
    c->uniform = uniform;
    c->width = new (std::nothrow) int[(size_t)L + 1];
    c->off_w = new (std::nothrow) size_t[(size_t)L + 1];
    c->off_h = new (std::nothrow) size_t[(size_t)L + 1];
    c->off_a = new (std::nothrow) size_t[(size_t)L + 2];
    if (!c->width || !c->off_w || !c->off_h || !c->off_a) {
        lf_destroy(c);
        return LF_ENOMEM;
    }
    c->off_w[0] = 0; c->off_h[0] = 0; c->off_a[0] = 0;
    for (int l = 0; l <= L; ++l) {
        c->width[l] = widths[l];
        c->off_a[l + 1] = c->off_a[l] + (size_t)widths[l];
        if (l >= 1) {
            c->off_w[l] = c->off_w[l - 1] + (size_t)widths[l] * (size_t)widths[l - 1];
            c->off_h[l] = c->off_h[l - 1] + (size_t)widths[l];
        }
    }
    if (uniform) {
        c->pk_N = N; c->pk_L = L;
    } else if (L >= 3) {
        bool hidden_equal = true;
        for (int l = 2; l <= L - 1; ++l) hidden_equal = hidden_equal && widths[l] == widths[1];
        if (hidden_equal) { c->pk_N = widths[1]; c->pk_L = L - 2; }
    }
    c->device = dev;
    c->sm_count = prop.multiProcessorCount;
    c->smem_optin = (int)prop.sharedMemPerBlockOptin;
    c->stream = nullptr;
    static const char* const variant_names[] = {"auto", "streams", "persistent", "fused"};
    static const char* const tiling_names[] = {"auto", "clusters", "columns"};
    c->opt_variant = option_from_env("LF_VARIANT", variant_names, 4, LF_VARIANT_AUTO);
    c->opt_fused_tiling = option_from_env("LF_FUSED_TILING", tiling_names, 3, LF_FUSED_TILING_AUTO);
    c->opt_gw_math = LF_GW_MATH_AUTO;
    c->wait_budget_us = 2000000;
    c->use_graph = 1;
    c->tc_pair_kernels = 1;
    c->shard_rank = 0; c->shard_count = 1;

    bool ok = true;
    size_t ws = 0;
    // scratch of the B = 1 delta matvec: (row chunks of w^{l+1}) x n_l partial sums, the largest layer
    size_t partial_floats = 4;
    for (int l = 1; l < L; ++l) {
        const size_t need = (size_t)lfk_delta_row_chunks(widths[l + 1]) * (size_t)widths[l];
        if (need > partial_floats) partial_floats = need;
    }
    size_t partial_bytes = partial_floats * sizeof(float);
    size_t counter_bytes = (size_t)(N / 128 + 1) * sizeof(unsigned);
    c->sync_words_count = lf_sync_words_needed(c);
    ok = ok && cudaMalloc(&c->partial, partial_bytes) == cudaSuccess; ws += partial_bytes;
    ok = ok && cudaMalloc(&c->counters, counter_bytes) == cudaSuccess; ws += counter_bytes;
    ok = ok && cudaMalloc(&c->sync_words, c->sync_words_count * sizeof(unsigned)) == cudaSuccess;
    ws += c->sync_words_count * sizeof(unsigned);
    ok = ok && cudaMalloc(&c->status_dev, sizeof(unsigned)) == cudaSuccess; ws += sizeof(unsigned);
    if (B > 1 && B <= lfk_small_batch_max()) {
        size_t sb_floats = 0;
        for (int l = 1; l < L; ++l) {
            const size_t f = lfk_delta_small_batch_scratch_floats(widths[l + 1], widths[l], B);
            if (f > sb_floats) sb_floats = f;
        }
        if (sb_floats) { ok = ok && cudaMalloc(&c->sb_partial, sb_floats * sizeof(float)) == cudaSuccess; ws += sb_floats * sizeof(float); }
    }
    const size_t dg_bytes = lf_delta_tc_scratch_bytes(c);
    if (dg_bytes) { ok = ok && cudaMalloc(&c->dg_partial, dg_bytes) == cudaSuccess; ws += dg_bytes; }
    ok = ok && cudaMallocHost(&c->status_host, sizeof(unsigned)) == cudaSuccess;
    if (ok) {
        ok = ok && cudaMemset(c->counters, 0, counter_bytes) == cudaSuccess;
        ok = ok && cudaMemset(c->sync_words, 0, c->sync_words_count * sizeof(unsigned)) == cudaSuccess;
        ok = ok && cudaMemset(c->status_dev, 0, sizeof(unsigned)) == cudaSuccess;
        *c->status_host = 0;
    }
    c->wstreams = new (std::nothrow) cudaStream_t[c->keff]();
    c->ready_ev = new (std::nothrow) cudaEvent_t[L]();
    c->done_ev = new (std::nothrow) cudaEvent_t[c->keff]();
    ok = ok && c->wstreams && c->ready_ev && c->done_ev;
    if (ok) {
        for (int j = 0; j < c->keff && ok; ++j) {
            ok = cudaStreamCreateWithFlags(&c->wstreams[j], cudaStreamNonBlocking) == cudaSuccess;
            ok = ok && cudaEventCreateWithFlags(&c->done_ev[j], cudaEventDisableTiming) == cudaSuccess;
        }
        for (int l = 0; l < L && ok; ++l)
            ok = cudaEventCreateWithFlags(&c->ready_ev[l], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->fork_ev, cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) {
        cudaError_t e = cudaGetLastError();
        bool oom = (e == cudaErrorMemoryAllocation);
        lf_destroy(c);
        return oom ? LF_ENOMEM : LF_ECUDA;
    }
    c->stats.L = L; c->stats.N = N; c->stats.B = B; c->stats.k = k;
    c->stats.k_effective = c->keff;
    c->stats.sm_count = c->sm_count;
    c->stats.workspace_bytes = (long long)ws;
    *out = c;
    return LF_OK;
}

int lf_set_stream(lf_ctx* ctx, void* cuda_stream)
{
    if (!ctx) return LF_ENULL;
    if (ctx->stream != (cudaStream_t)cuda_stream) drop_graph(ctx);
    ctx->stream = (cudaStream_t)cuda_stream;
    return LF_OK;
}

int lf_set_option(lf_ctx* ctx, int key, long long value)
{
    if (!ctx) return LF_ENULL;
    switch (key) {
        case LF_OPT_VARIANT:
            if (value < LF_VARIANT_AUTO || value > LF_VARIANT_FUSED) return LF_EINVAL;
            ctx->opt_variant = (int)value;
            return LF_OK;
        case LF_OPT_GW_MATH:
            if (value < LF_GW_MATH_AUTO || value > LF_GW_MATH_TF32) return LF_EINVAL;
            ctx->opt_gw_math = (int)value;
            return LF_OK;
        case LF_OPT_WAIT_BUDGET_US:
            if (value < 1 || value > 60000000LL) return LF_EINVAL;
            ctx->wait_budget_us = value;
            return LF_OK;
        case LF_OPT_DELTA_MATH:
            if (value < LF_DELTA_MATH_AUTO || value > LF_DELTA_MATH_TF32_BF16) return LF_EINVAL;
            ctx->opt_delta_math = (int)value;
            return LF_OK;
        case LF_OPT_TC_TILING:
            if (value < LF_TC_TILING_AUTO || value > LF_TC_TILING_TWO_SM) return LF_EINVAL;
            ctx->tc_pair_kernels = value != LF_TC_TILING_ONE_SM;
            drop_graph(ctx);
            return LF_OK;
        case LF_OPT_COST:
            if (value != LF_COST_QUADRATIC && value != LF_COST_CROSS_ENTROPY) return LF_EINVAL;
            ctx->opt_cost = (int)value;
            return LF_OK;
        case LF_OPT_ACTIVATION:
            if (value < LF_ACT_SIGMOID || value > LF_ACT_RELU) return LF_EINVAL;
            ctx->opt_act = (int)value;
            return LF_OK;
        case LF_OPT_SHARD_COUNT:
            if (value < 1 || value > 65535) return LF_EINVAL;
            ctx->shard_count = (int)value;
            ctx->shard_rank = 0;
            return LF_OK;
        case LF_OPT_SHARD_RANK:
            if (value < 0 || value >= ctx->shard_count) return LF_EINVAL;
            ctx->shard_rank = (int)value;
            return LF_OK;
        case LF_OPT_FUSED_TILING:
            if (value < LF_FUSED_TILING_AUTO || value > LF_FUSED_TILING_COLUMNS) return LF_EINVAL;
            ctx->opt_fused_tiling = (int)value;
            return LF_OK;
        case LF_OPT_TIME_CALLS:
            if (value != 0 && value != 1) return LF_EINVAL;
            if (value && !ctx->t_begin_ev) {
                cudaEvent_t b = nullptr, e = nullptr;
                if (cudaEventCreate(&b) != cudaSuccess || cudaEventCreate(&e) != cudaSuccess) {
                    if (b) cudaEventDestroy(b);
                    ctx->last_cuda_error = (int)cudaGetLastError();
                    return LF_ECUDA;
                }
                ctx->t_begin_ev = b; ctx->t_end_ev = e;
            }
            ctx->time_calls = (int)value;
            return LF_OK;
        case LF_OPT_WITHHOLD:
            if (value < 0 || value > 2) return LF_EINVAL;
            ctx->withhold = (int)value;
            return LF_OK;
        case LF_OPT_USE_GRAPH:
            if (value != 0 && value != 1) return LF_EINVAL;
            ctx->use_graph = (int)value;
            if (!value) drop_graph(ctx);
            return LF_OK;
        default:
            return LF_EINVAL;
    }
}

int lf_forward(lf_ctx* ctx, const float* w, const float* b, const float* x, float* z, float* a)
{
    if (!ctx) return LF_ENULL;
    const void* ps[] = {w, b, x, z, a};
    int rc = check_ptrs(ps, 5);
    if (rc != LF_OK) return rc;
    const int L = ctx->L, B = ctx->B;
    cudaStream_t s = ctx->stream;
    int launches = 0;
    if (a != x) LF_CUDA_TRY(ctx, lfk_copy_input(x, a, (size_t)B * ctx->width[0], s));  // Eq. x
    for (int l = 1; l <= L; ++l) {
        const float* w_l = w + w_at(ctx, l);
        const float* b_l = b + v_at(ctx, l);
        const float* a_prev = a + a_at(ctx, l - 1);
        float* z_l = z + h_at(ctx, l);
        float* a_l = a + a_at(ctx, l);
        const int n_out = ctx->width[l], n_in = ctx->width[l - 1];
        if (B == 1) {
            LF_CUDA_TRY(ctx, lfk_forward_matvec(w_l, b_l, a_prev, z_l, a_l, n_out, n_in, ctx->opt_act, s));
            ++launches;
        } else if (resolve_forward_math(ctx) >= LF_DELTA_MATH_3XTF32) {
            int rc2 = lf_forward_gemm_tc(ctx, w_l, b_l, a_prev, z_l, a_l, n_out, n_in, resolve_forward_math(ctx), s, &launches);
            if (rc2 != LF_OK) return rc2;
        } else {
            LF_CUDA_TRY(ctx, lfk_forward_gemm(w_l, b_l, a_prev, z_l, a_l, n_out, n_in, B, ctx->opt_act, s));
            ++launches;
        }
    }
    ctx->stats.launches_forward = launches;
    ctx->stats.activation = ctx->opt_act;
    return LF_OK;
}

// LF_OPT_TIME_CALLS: events around a backward call on the context's stream (not during a capture
// the caller may have open on it: an event recorded there could not be read back).
struct call_timer {
    lf_ctx* c;
    bool on;
    explicit call_timer(lf_ctx* ctx) : c(ctx), on(false)
    {
        if (!c->time_calls || !c->t_begin_ev) return;
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(c->stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
            cudaGetLastError();
            return;
        }
        on = cudaEventRecord(c->t_begin_ev, c->stream) == cudaSuccess;
    }
    void done(int rc)
    {
        if (on && rc == LF_OK && cudaEventRecord(c->t_end_ev, c->stream) == cudaSuccess) c->timed_call_pending = true;
    }
};

static int backward_impl(lf_ctx* ctx, const float* w, const float* z, const float* a, const float* y,
                         float* delta, float* gw, float* gb)
{
    int variant = resolve_variant(ctx);
    const int gw_math = resolve_gw_math(ctx);
    const bool widths_single_launch = !ctx->uniform && variant == LF_VARIANT_FUSED &&
                                      ctx->opt_fused_tiling != LF_FUSED_TILING_CLUSTERS && lf_columns_widths_supported(ctx);
    if (variant != LF_VARIANT_STREAMS && !widths_single_launch && !lf_persistent_supported(ctx, variant))
        variant = LF_VARIANT_STREAMS;
    ctx->stats.variant = variant;
    ctx->stats.gw_math = gw_math;
    ctx->stats.delta_math = resolve_delta_math(ctx);
    ctx->stats.cost = ctx->opt_cost;
    ctx->stats.activation = ctx->opt_act;
    ctx->stats.shard_rank = ctx->shard_rank; ctx->stats.shard_count = ctx->shard_count;
    ctx->stats.fused_tiling = 0;
    if (variant == LF_VARIANT_STREAMS)
        return backward_streams(ctx, w, z, a, y, delta, gw, gb, gw_math);
    if (ctx->uniform)
        return lf_backward_persistent(ctx, variant, w, a, y, delta, gw, gb, ctx->sgd_w, 0, 0);
    if (variant == LF_VARIANT_FUSED && ctx->opt_fused_tiling != LF_FUSED_TILING_CLUSTERS && lf_columns_widths_supported(ctx))
        return lf_backward_columns_widths(ctx, w, a, y, delta, gw, gb, ctx->sgd_w);
    return backward_hidden_run(ctx, variant, w, a, y, delta, gw, gb, gw_math);
}

int lf_backward(lf_ctx* ctx, const float* w, const float* z, const float* a, const float* y,
                float* delta, float* gw, float* gb)
{
    if (!ctx) return LF_ENULL;
    const void* ps[] = {w, z, a, y, delta, gw, gb};
    int rc = check_ptrs(ps, 7);
    if (rc != LF_OK) return rc;
    if (ctx->opt_cost == LF_COST_CROSS_ENTROPY && ctx->opt_act != LF_ACT_SIGMOID) return LF_EINVAL;
    call_timer timer(ctx);
    rc = backward_impl(ctx, w, z, a, y, delta, gw, gb);
    timer.done(rc);
    return rc;
}

int lf_grad_w(lf_ctx* ctx, const float* delta_l, const float* a_prev, float* gw_l)
{
    if (!ctx) return LF_ENULL;
    const void* ps[] = {delta_l, a_prev, gw_l};
    int rc = check_ptrs(ps, 3);
    if (rc != LF_OK) return rc;
    if (!ctx->uniform) return LF_EINVAL;   // the call names no layer, so it cannot know that layer's shape
    const int gw_math = resolve_gw_math(ctx);
    ctx->stats.gw_math = gw_math;
    const lf_sgd plain = {nullptr, 0.f};
    int launches = 0;
    if (ctx->B == 1)
        LF_CUDA_TRY(ctx, lfk_gw_rank1(delta_l, a_prev, gw_l, ctx->N, ctx->N, plain, ctx->stream));
    else if (gw_math == LF_GW_MATH_TF32)
        return lf_gw_gemm_tf32(ctx, delta_l, a_prev, gw_l, ctx->N, ctx->N, plain, ctx->stream, &launches);
    else
        LF_CUDA_TRY(ctx, lfk_gw_gemm_fp32(delta_l, a_prev, gw_l, ctx->N, ctx->N, ctx->B, plain, ctx->stream));
    return LF_OK;
}

int lf_backward_sgd(lf_ctx* ctx, const float* w, const float* z, const float* a, const float* y,
                    float eta, float* delta, float* w_new, float* gb)
{
    if (!ctx) return LF_ENULL;
    if (!w || !w_new) return LF_ENULL;
    if (!(eta == eta) || eta - eta != 0.f) return LF_EINVAL;          // NaN or infinite
    const size_t bytes = ctx->off_w[ctx->L] * sizeof(float);
    const char* lo = reinterpret_cast<const char*>(w);
    const char* out = reinterpret_cast<const char*>(w_new);
    if (out < lo + bytes && lo < out + bytes) return LF_EINVAL;        // w_new overlaps w
    ctx->sgd_on = 1; ctx->sgd_eta = eta; ctx->sgd_w = w;
    const int rc = lf_backward(ctx, w, z, a, y, delta, w_new, gb);
    ctx->sgd_on = 0; ctx->sgd_w = nullptr;
    return rc;
}

int lf_backward_host(lf_ctx* ctx, const float* w, const float* z, const float* a, const float* y,
                     float* delta, float* gw, float* gb)
{
    if (!ctx) return LF_ENULL;
    const void* ps[] = {w, z, a, y, delta, gw, gb};
    for (int i = 0; i < 7; ++i)
        if (!ps[i]) return LF_ENULL;
    if (ctx->opt_cost == LF_COST_CROSS_ENTROPY && ctx->opt_act != LF_ACT_SIGMOID) return LF_EINVAL;
    const int Li = ctx->L;
    const size_t Bs = (size_t)ctx->B;
    // staging layout, every block a multiple of 4 floats: w | a | y | delta | gw | gb  (z stays on the
    // host: no kernel of the backward pass reads it, sigma' comes from a)
    const size_t n_w = ctx->off_w[Li], n_a = Bs * ctx->off_a[Li + 1], n_y = Bs * (size_t)ctx->width[Li],
                 n_d = Bs * ctx->off_h[Li], n_gw = n_w, n_gb = ctx->off_h[Li];
    const size_t total = n_w + n_a + n_y + n_d + n_gw + n_gb;
    if (!ctx->stage) {
        cudaError_t e = cudaMalloc(&ctx->stage, total * sizeof(float));
        if (e != cudaSuccess) {
            ctx->stage = nullptr;
            ctx->last_cuda_error = (int)e;
            cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? LF_ENOMEM : LF_ECUDA;
        }
        ctx->stage_bytes = total * sizeof(float);
        ctx->stats.workspace_bytes += (long long)ctx->stage_bytes;
    }
    float* d_w = ctx->stage;
    float* d_a = d_w + n_w;
    float* d_y = d_a + n_a;
    float* d_d = d_y + n_y;
    float* d_gw = d_d + n_d;
    float* d_gb = d_gw + n_gw;
    // copy streams and per-layer arrival events, created on first use: everything is built first and
    // handed to the context only when all of it exists, so a failure half way leaves nothing behind
    // that a later call would take for a finished set-up
    if (!ctx->host_path_ready) {
        cudaStream_t hs = nullptr, ds = nullptr;
        cudaEvent_t* w_ev = new (std::nothrow) cudaEvent_t[Li]();
        cudaEvent_t* g_ev = new (std::nothrow) cudaEvent_t[Li]();
        cudaEvent_t one[3] = {nullptr, nullptr, nullptr};
        bool ok = w_ev && g_ev;
        cudaError_t e = cudaSuccess;
        if (ok) {
            ok = (e = cudaStreamCreateWithFlags(&hs, cudaStreamNonBlocking)) == cudaSuccess &&
                 (e = cudaStreamCreateWithFlags(&ds, cudaStreamNonBlocking)) == cudaSuccess;
            for (int l = 0; l < Li && ok; ++l)
                ok = (e = cudaEventCreateWithFlags(&w_ev[l], cudaEventDisableTiming)) == cudaSuccess &&
                     (e = cudaEventCreateWithFlags(&g_ev[l], cudaEventDisableTiming)) == cudaSuccess;
            for (int i = 0; i < 3 && ok; ++i)
                ok = (e = cudaEventCreateWithFlags(&one[i], cudaEventDisableTiming)) == cudaSuccess;
        }
        if (!ok) {
            const bool no_host_memory = !w_ev || !g_ev;
            for (int l = 0; l < Li; ++l) {
                if (w_ev && w_ev[l]) cudaEventDestroy(w_ev[l]);
                if (g_ev && g_ev[l]) cudaEventDestroy(g_ev[l]);
            }
            for (int i = 0; i < 3; ++i)
                if (one[i]) cudaEventDestroy(one[i]);
            if (hs) cudaStreamDestroy(hs);
            if (ds) cudaStreamDestroy(ds);
            delete[] w_ev;
            delete[] g_ev;
            cudaGetLastError();
            if (no_host_memory) return LF_ENOMEM;
            ctx->last_cuda_error = (int)e;
            return LF_ECUDA;
        }
        ctx->h2d_stream = hs; ctx->d2h_stream = ds;
        ctx->w_ready_ev = w_ev; ctx->gw_done_ev = g_ev;
        ctx->small_ev = one[0]; ctx->h2d_done_ev = one[1]; ctx->d2h_done_ev = one[2];
        ctx->host_path_ready = true;
    }
    // The copies are pipelined with the per-layer schedule: the weights arrive top layer
    // first on a copy stream, the chain step of layer l starts as soon as w^{l+1} is there,
    // and gw^l is sent back as soon as its worker has written it, so the two PCIe directions
    // are busy at the same time.  All downloads go through ONE stream, in layer order: spread
    // over the k worker streams they ran 10-14 % slower (measured at L = 32, N = 1024).
    cudaStream_t s = ctx->stream, hs = ctx->h2d_stream, ds = ctx->d2h_stream;
    const int gw_math = resolve_gw_math(ctx);
    ctx->stats.variant = LF_VARIANT_STREAMS;
    ctx->stats.gw_math = gw_math;
    ctx->stats.delta_math = resolve_delta_math(ctx);
    ctx->stats.cost = ctx->opt_cost;
    ctx->stats.activation = ctx->opt_act;
    ctx->stats.shard_rank = ctx->shard_rank; ctx->stats.shard_count = ctx->shard_count;
    ctx->stats.fused_tiling = 0;
    int launches = 0;
    call_timer timer(ctx);
    LF_CUDA_TRY(ctx, cudaEventRecord(ctx->fork_ev, s));
    // From here on the copy, download and worker streams are forked off the context's stream: whatever
    // goes wrong below, they are joined back into it before the call returns (`fail` keeps the
    // first error; the remaining enqueues are skipped).
    int fail = LF_OK;
    auto tried = [&](cudaError_t e) {
        if (e != cudaSuccess && fail == LF_OK) { ctx->last_cuda_error = (int)e; fail = LF_ECUDA; }
        return fail == LF_OK;
    };
    tried(cudaStreamWaitEvent(hs, ctx->fork_ev, 0));
    tried(cudaStreamWaitEvent(ds, ctx->fork_ev, 0));
    for (int j = 0; j < ctx->keff; ++j) tried(cudaStreamWaitEvent(ctx->wstreams[j], ctx->fork_ev, 0));
    if (fail == LF_OK) {
        tried(cudaMemcpyAsync(d_a, a, n_a * sizeof(float), cudaMemcpyHostToDevice, hs));
        tried(cudaMemcpyAsync(d_y, y, n_y * sizeof(float), cudaMemcpyHostToDevice, hs));
        tried(cudaEventRecord(ctx->small_ev, hs));
    }
    for (int l = Li; l >= 2 && fail == LF_OK; --l) {   // w^1 is never read: Eq. bp2 needs w^{l+1} for l = L-1 .. 1
        const size_t M = (size_t)ctx->width[l] * (size_t)ctx->width[l - 1];
        tried(cudaMemcpyAsync(d_w + w_at(ctx, l), w + w_at(ctx, l), M * sizeof(float), cudaMemcpyHostToDevice, hs));
        tried(cudaEventRecord(ctx->w_ready_ev[l - 1], hs));
    }
    if (fail == LF_OK) tried(cudaStreamWaitEvent(s, ctx->small_ev, 0));
    for (int l = Li; l >= 1 && fail == LF_OK; --l) {
        if (l < Li && !tried(cudaStreamWaitEvent(s, ctx->w_ready_ev[l], 0))) break;   // w^{l+1}
        int rc = enqueue_chain_step(ctx, l, d_w, d_a, d_y, d_d, d_gb, s, &launches);
        if (rc != LF_OK) { fail = rc; break; }
        if (!lf_layer_owned(ctx, l)) continue;    // another shard's layer: nothing to compute or send back
        const int j = lf_layer_worker(ctx, l);
        cudaStream_t wsj = ctx->wstreams[j];
        if (!tried(cudaEventRecord(ctx->ready_ev[l - 1], s)) ||
            !tried(cudaStreamWaitEvent(wsj, ctx->ready_ev[l - 1], 0)))
            break;
        rc = enqueue_gradients(ctx, l, d_a, d_d, d_gw, d_gb, gw_math, wsj, &launches);
        if (rc != LF_OK) { fail = rc; break; }
        const size_t M = (size_t)ctx->width[l] * (size_t)ctx->width[l - 1];
        tried(cudaEventRecord(ctx->gw_done_ev[l - 1], wsj));
        tried(cudaStreamWaitEvent(ds, ctx->gw_done_ev[l - 1], 0));
        tried(cudaMemcpyAsync(gw + w_at(ctx, l), d_gw + w_at(ctx, l), M * sizeof(float), cudaMemcpyDeviceToHost, ds));
    }
    if (fail == LF_OK) {
        // the download stream has waited for the gw and gb of every layer done here; the end of the
        // chain (delta^1, the last thing written on s) it waits for explicitly
        tried(cudaEventRecord(ctx->small_ev, s));
        tried(cudaStreamWaitEvent(ds, ctx->small_ev, 0));
        tried(cudaMemcpyAsync(delta, d_d, n_d * sizeof(float), cudaMemcpyDeviceToHost, ds));
        if (ctx->B == 1 || ctx->shard_count == 1) {
            tried(cudaMemcpyAsync(gb, d_gb, n_gb * sizeof(float), cudaMemcpyDeviceToHost, ds));
        } else {
            for (int l = 1; l <= Li; ++l)     // B > 1: gb^l exists only for this shard's layers
                if (lf_layer_owned(ctx, l))
                    tried(cudaMemcpyAsync(gb + v_at(ctx, l), d_gb + v_at(ctx, l),
                                          (size_t)ctx->width[l] * sizeof(float), cudaMemcpyDeviceToHost, ds));
        }
    }
    // join: on every path, also after a failure
    cudaError_t je = cudaEventRecord(ctx->d2h_done_ev, ds);
    if (je == cudaSuccess) je = cudaEventRecord(ctx->h2d_done_ev, hs);
    for (int j = 0; j < ctx->keff && je == cudaSuccess; ++j) {
        je = cudaEventRecord(ctx->done_ev[j], ctx->wstreams[j]);
        if (je == cudaSuccess) je = cudaStreamWaitEvent(s, ctx->done_ev[j], 0);
    }
    if (je == cudaSuccess) je = cudaStreamWaitEvent(s, ctx->h2d_done_ev, 0);
    if (je == cudaSuccess) je = cudaStreamWaitEvent(s, ctx->d2h_done_ev, 0);
    if (je != cudaSuccess && fail == LF_OK) { ctx->last_cuda_error = (int)je; fail = LF_ECUDA; }
    ctx->stats.launches_backward = launches;
    timer.done(fail);
    return fail;
}

int lf_sync(lf_ctx* ctx)
{
    if (!ctx) return LF_ENULL;
    LF_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->status_host, ctx->status_dev, sizeof(unsigned),
                                     cudaMemcpyDeviceToHost, ctx->stream));
    LF_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
    if (ctx->timed_call_pending) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ctx->t_begin_ev, ctx->t_end_ev) == cudaSuccess) ctx->stats.last_backward_ms = ms;
        else cudaGetLastError();
        ctx->timed_call_pending = false;
    }
    unsigned st = *ctx->status_host;
    ctx->stats.device_status = st;
    if (st != 0) {
        cudaMemsetAsync(ctx->status_dev, 0, sizeof(unsigned), ctx->stream);  // next call starts clean
        if (st & (LF_DEV_TIMEOUT_FLAG | LF_DEV_TIMEOUT_BARRIER)) return LF_ETIMEOUT;
        return LF_EINVAL;
    }
    return LF_OK;
}

int lf_owner(const lf_ctx* ctx, int l)
{
    if (!ctx || l < 1 || l > ctx->L) return -1;
    return lf_layer_owned(ctx, l) ? lf_layer_worker(ctx, l) : -1;
}

int lf_get_stats(lf_ctx* ctx, lf_stats* out)
{
    if (!ctx || !out) return LF_ENULL;
    *out = ctx->stats;
    return LF_OK;
}

int lf_last_cuda_error(const lf_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int lf_destroy(lf_ctx* ctx)
{
    if (!ctx) return LF_ENULL;
    cudaStreamSynchronize(ctx->stream);
    drop_graph(ctx);
    if (ctx->wstreams) {
        for (int j = 0; j < ctx->keff; ++j)
            if (ctx->wstreams[j]) { cudaStreamSynchronize(ctx->wstreams[j]); cudaStreamDestroy(ctx->wstreams[j]); }
        delete[] ctx->wstreams;
    }
    if (ctx->done_ev) {
        for (int j = 0; j < ctx->keff; ++j)
            if (ctx->done_ev[j]) cudaEventDestroy(ctx->done_ev[j]);
        delete[] ctx->done_ev;
    }
    if (ctx->ready_ev) {
        for (int l = 0; l < ctx->L; ++l)
            if (ctx->ready_ev[l]) cudaEventDestroy(ctx->ready_ev[l]);
        delete[] ctx->ready_ev;
    }
    if (ctx->fork_ev) cudaEventDestroy(ctx->fork_ev);
    if (ctx->partial) cudaFree(ctx->partial);
    if (ctx->counters) cudaFree(ctx->counters);
    if (ctx->sync_words) cudaFree(ctx->sync_words);
    if (ctx->status_dev) cudaFree(ctx->status_dev);
    if (ctx->dg_partial) cudaFree(ctx->dg_partial);
    if (ctx->sb_partial) cudaFree(ctx->sb_partial);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    if (ctx->stage) cudaFree(ctx->stage);
    if (ctx->h2d_stream) { cudaStreamSynchronize(ctx->h2d_stream); cudaStreamDestroy(ctx->h2d_stream); }
    if (ctx->d2h_stream) { cudaStreamSynchronize(ctx->d2h_stream); cudaStreamDestroy(ctx->d2h_stream); }
    if (ctx->gw_done_ev) {
        for (int l = 0; l < ctx->L; ++l)
            if (ctx->gw_done_ev[l]) cudaEventDestroy(ctx->gw_done_ev[l]);
        delete[] ctx->gw_done_ev;
    }
    if (ctx->d2h_done_ev) cudaEventDestroy(ctx->d2h_done_ev);
    delete[] ctx->width;
    delete[] ctx->off_w;
    delete[] ctx->off_h;
    delete[] ctx->off_a;
    if (ctx->w_ready_ev) {
        for (int l = 0; l < ctx->L; ++l)
            if (ctx->w_ready_ev[l]) cudaEventDestroy(ctx->w_ready_ev[l]);
        delete[] ctx->w_ready_ev;
    }
    if (ctx->t_begin_ev) cudaEventDestroy(ctx->t_begin_ev);
    if (ctx->t_end_ev) cudaEventDestroy(ctx->t_end_ev);
    if (ctx->small_ev) cudaEventDestroy(ctx->small_ev);
    if (ctx->h2d_done_ev) cudaEventDestroy(ctx->h2d_done_ev);
    lf_persistent_release(ctx);
    lf_columns_release(ctx);
    lf_tf32_release(ctx);
    delete ctx;
    return LF_OK;
}

}  // extern "C"
