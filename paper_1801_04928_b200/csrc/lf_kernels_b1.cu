// Single-sample (B = 1) kernels, one launch per layer: the forward matvec (Eq. z, Eq. a),
// the output error (Eq. bp1), the transposed matvec of the delta recurrence (Eq. bp2) and the
// rank-1 weight-gradient writer (Eq. bp4).  All are HBM-bound streams over one layer's matrix
// (n_out x n_in, row-major; square when all layers have one width):
// 128-bit accesses, rows walked in the order they sit in memory.
#include <mutex>

#include "lf_internal.h"

namespace {

__device__ __forceinline__ float4 ld_stream(const float4* p)
{
    // Weights are read once per pass: keep them from displacing the vectors in L1.
    return __ldcs(p);
}

// ---- Eq. z, Eq. a : z_j = sum_k w_jk a_k + b_j ; a_j = sigma(z_j).  One warp per row. ---------
constexpr int FWD_WARPS = 8;

__global__ void __launch_bounds__(FWD_WARPS * 32)
k_forward_matvec(const float* __restrict__ w, const float* __restrict__ b,
                 const float* __restrict__ a_prev, float* __restrict__ z,
                 float* __restrict__ a, int n_out, int n_in, int act)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * FWD_WARPS + warp;
    if (j >= n_out) return;
    const float4* wr = reinterpret_cast<const float4*>(w + (size_t)j * n_in);
    const float4* av = reinterpret_cast<const float4*>(a_prev);
    const int n4 = n_in >> 2;
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    int c = lane;
    for (; c + 96 < n4; c += 128) {  // four independent 128-bit loads in flight per lane
        float4 w0 = ld_stream(wr + c), w1 = ld_stream(wr + c + 32);
        float4 w2 = ld_stream(wr + c + 64), w3 = ld_stream(wr + c + 96);
        float4 a0 = av[c], a1 = av[c + 32], a2 = av[c + 64], a3 = av[c + 96];
        acc0 = fmaf(w0.x, a0.x, fmaf(w0.y, a0.y, fmaf(w0.z, a0.z, fmaf(w0.w, a0.w, acc0))));
        acc1 = fmaf(w1.x, a1.x, fmaf(w1.y, a1.y, fmaf(w1.z, a1.z, fmaf(w1.w, a1.w, acc1))));
        acc2 = fmaf(w2.x, a2.x, fmaf(w2.y, a2.y, fmaf(w2.z, a2.z, fmaf(w2.w, a2.w, acc2))));
        acc3 = fmaf(w3.x, a3.x, fmaf(w3.y, a3.y, fmaf(w3.z, a3.z, fmaf(w3.w, a3.w, acc3))));
    }
    for (; c < n4; c += 32) {
        float4 w0 = ld_stream(wr + c);
        float4 a0 = av[c];
        acc0 = fmaf(w0.x, a0.x, fmaf(w0.y, a0.y, fmaf(w0.z, a0.z, fmaf(w0.w, a0.w, acc0))));
    }
    float acc = (acc0 + acc1) + (acc2 + acc3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
        float zz = acc + b[j];
        z[j] = zz;
        a[j] = lf_act(zz, act);
    }
}

// ---- Eq. bp1 : delta^L = grad_a C (.) sigma'(z^L), sigma' = a (1 - a) ---------------------------
// quadratic cost: grad_a C = a^L - y;  cross-entropy: grad_a C = (a^L - y) / (a^L (1 - a^L)), which
// the factor sigma' cancels, leaving delta^L = a^L - y
__global__ void k_output_error(const float* __restrict__ aL, const float* __restrict__ y,
                               float* __restrict__ deltaL, float* __restrict__ gbL, size_t n, int cost, int act)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float av = aL[i];
    float d = av - y[i];
    if (cost == LF_COST_QUADRATIC) d *= lf_act_prime(av, act);
    deltaL[i] = d;
    if (gbL) gbL[i] = d;  // Eq. bp3 for a single sample
}

// ---- Eq. bp2 : delta^l_k = (sum_j w^{l+1}_jk delta^{l+1}_j) sigma'(z^l_k) ------------------------
// A column reduction over a row-major matrix.  The grid is (column strips) x (row chunks); a
// CTA walks its rows with every lane owning four adjacent columns, so each warp reads 512
// contiguous bytes of a row.  Partial sums go to scratch; the CTA that arrives last at a strip
// adds the chunks in a fixed order (so results do not depend on scheduling), applies sigma'
// and writes delta^l (= grad_b^l).
constexpr int DMV_WARPS = 8;
constexpr int DMV_STRIP4 = 32;  // float4 columns per strip (128 floats)

__host__ __device__ inline int dmv_rows_per_chunk(int n_up) { return n_up <= 2048 ? 32 : 64; }

__global__ void __launch_bounds__(DMV_WARPS * 32)
k_delta_matvec(const float* __restrict__ w_up, const float* __restrict__ delta_up,
               const float* __restrict__ a_l, float* __restrict__ delta_l,
               float* __restrict__ gb_l, float* __restrict__ partial,
               unsigned* __restrict__ counters, int n_up, int n_l, int rows_per_chunk, int chunks, int act)
{
    // w_up is n_up x n_l: rows = neurons j of layer l+1, columns = neurons k of layer l
    __shared__ float4 red[DMV_WARPS][DMV_STRIP4];
    __shared__ bool is_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int strip = blockIdx.x, chunk = blockIdx.y;
    const int n4 = n_l >> 2;
    const int c4 = strip * DMV_STRIP4 + lane;
    const bool col_ok = c4 < n4;
    const int r0 = chunk * rows_per_chunk;
    const int r1 = min(n_up, r0 + rows_per_chunk);

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col_ok) {
        const float4* wp = reinterpret_cast<const float4*>(w_up) + c4;
#pragma unroll 4
        for (int r = r0 + warp; r < r1; r += DMV_WARPS) {
            float4 wv = ld_stream(wp + (size_t)r * n4);
            float d = delta_up[r];
            acc.x = fmaf(wv.x, d, acc.x);
            acc.y = fmaf(wv.y, d, acc.y);
            acc.z = fmaf(wv.z, d, acc.z);
            acc.w = fmaf(wv.w, d, acc.w);
        }
    }
    red[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && col_ok) {
        float4 s = red[0][lane];
#pragma unroll
        for (int q = 1; q < DMV_WARPS; ++q) {
            float4 t = red[q][lane];
            s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
        }
        reinterpret_cast<float4*>(partial)[(size_t)chunk * n4 + c4] = s;
        __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned prev = atomicAdd(&counters[strip], 1u);
        is_last = (prev == (unsigned)chunks - 1u);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // Last CTA of this strip: warp q adds chunks q, q+8, ... ; warp 0 then adds the 8 sums.
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col_ok) {
        for (int q = warp; q < chunks; q += DMV_WARPS) {
            float4 t = __ldcg(reinterpret_cast<const float4*>(partial) + (size_t)q * n4 + c4);
            s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
        }
    }
    __syncthreads();
    red[warp][lane] = s;
    __syncthreads();
    if (warp == 0 && col_ok) {
        float4 t0 = red[0][lane];
#pragma unroll
        for (int q = 1; q < DMV_WARPS; ++q) {
            float4 t = red[q][lane];
            t0.x += t.x; t0.y += t.y; t0.z += t.z; t0.w += t.w;
        }
        float4 av = reinterpret_cast<const float4*>(a_l)[c4];
        float4 d;
        d.x = t0.x * lf_act_prime(av.x, act);
        d.y = t0.y * lf_act_prime(av.y, act);
        d.z = t0.z * lf_act_prime(av.z, act);
        d.w = t0.w * lf_act_prime(av.w, act);
        reinterpret_cast<float4*>(delta_l)[c4] = d;
        if (gb_l) reinterpret_cast<float4*>(gb_l)[c4] = d;  // Eq. bp3
    }
    if (threadIdx.x == 0) counters[strip] = 0u;  // ready for the next launch
}

// ---- Eq. bp4 : gw_jk = delta_j a_k.  A pure store stream: one multiply per stored element. ----
constexpr int GW1_THREADS = 256;

__global__ void __launch_bounds__(GW1_THREADS)
k_gw_rank1(const float* __restrict__ delta_l, const float* __restrict__ a_prev,
           float* __restrict__ gw_l, int n_out, int n_in, const lf_sgd sgd)
{
    const int n4 = n_in >> 2;
    const size_t total4 = (size_t)n_out * n4;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    float4* out = reinterpret_cast<float4*>(gw_l);
    const float4* av = reinterpret_cast<const float4*>(a_prev);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total4; i += stride) {
        int j = (int)(i / n4);
        int c = (int)(i - (size_t)j * n4);
        float d = delta_l[j];
        float4 a4 = av[c];
        float4 g = make_float4(d * a4.x, d * a4.y, d * a4.z, d * a4.w);
        if (sgd.w_sub)   // fused update: w - eta * g, the weights streamed through once
            g = lf_sgd_apply4(sgd.eta, ld_stream(reinterpret_cast<const float4*>(sgd.w_sub) + i), g);
        __stcs(out + i, g);
    }
}

}  // namespace

cudaError_t lfk_forward_matvec(const float* w_l, const float* b_l, const float* a_prev,
                               float* z_l, float* a_l, int n_out, int n_in, int act, cudaStream_t s)
{
    int grid = (n_out + FWD_WARPS - 1) / FWD_WARPS;
    k_forward_matvec<<<grid, FWD_WARPS * 32, 0, s>>>(w_l, b_l, a_prev, z_l, a_l, n_out, n_in, act);
    return cudaGetLastError();
}

cudaError_t lfk_copy_input(const float* x, float* a0, size_t n, cudaStream_t s)
{
    return cudaMemcpyAsync(a0, x, n * sizeof(float), cudaMemcpyDeviceToDevice, s);
}

cudaError_t lfk_output_error(const float* aL, const float* y, float* deltaL, float* gbL, int N,
                             int B, int cost, int act, cudaStream_t s)
{
    size_t n = (size_t)N * B;
    int grid = (int)((n + 255) / 256);
    k_output_error<<<grid, 256, 0, s>>>(aL, y, deltaL, B == 1 ? gbL : nullptr, n, cost, act);
    return cudaGetLastError();
}

int lfk_delta_row_chunks(int n_up)
{
    int r = dmv_rows_per_chunk(n_up);
    return (n_up + r - 1) / r;
}

cudaError_t lfk_delta_matvec(const float* w_up, const float* delta_up, const float* a_l,
                             float* delta_l, float* gb_l, float* partial, unsigned* counters,
                             int n_up, int n_l, int act, cudaStream_t s)
{
    int n4 = n_l >> 2;
    int strips = (n4 + DMV_STRIP4 - 1) / DMV_STRIP4;
    int rows = dmv_rows_per_chunk(n_up);
    int chunks = (n_up + rows - 1) / rows;
    dim3 grid(strips, chunks);
    k_delta_matvec<<<grid, DMV_WARPS * 32, 0, s>>>(w_up, delta_up, a_l, delta_l, gb_l, partial,
                                                  counters, n_up, n_l, rows, chunks, act);
    return cudaGetLastError();
}

cudaError_t lfk_gw_rank1(const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                         lf_sgd sgd, cudaStream_t s)
{
    size_t total4 = (size_t)n_out * (n_in >> 2);
    size_t want = (total4 + GW1_THREADS - 1) / GW1_THREADS;
    int grid = (int)(want < (size_t)148 * 16 ? want : (size_t)148 * 16);
    if (grid < 1) grid = 1;
    k_gw_rank1<<<grid, GW1_THREADS, 0, s>>>(delta_l, a_prev, gw_l, n_out, n_in, sgd);
    return cudaGetLastError();
}

// ---- Eq. bp2 for callers that must not allocate -------------------------------------------------
// The scratch of k_delta_matvec (partial column sums, then the per-strip arrival counters) lives
// in a file-scope device array instead of a context's workspace.  Every GPU that loads this
// library carries these LF_STATIC_SCRATCH_WORDS * 4 bytes (a little over 1 MiB) until exit.
namespace {

constexpr int LF_STATIC_MAX_N = 4096;                 // largest width the array is sized for
constexpr int LF_STATIC_MAX_CHUNKS = 64;              // row chunks never exceed this for N <= 4096
constexpr int LF_STATIC_COUNTER_WORDS = 64;           // >= column strips (N / 128) for N <= 4096
constexpr int LF_STATIC_PARTIAL_WORDS = LF_STATIC_MAX_CHUNKS * LF_STATIC_MAX_N;
constexpr int LF_STATIC_SCRATCH_WORDS = LF_STATIC_PARTIAL_WORDS + LF_STATIC_COUNTER_WORDS;

static __device__ __align__(256) float lf_static_scratch[LF_STATIC_SCRATCH_WORDS];

constexpr int LF_STATIC_MAX_DEVICES = 64;
std::mutex g_static_mutex;
float* g_static_scratch_addr[LF_STATIC_MAX_DEVICES];  // device address of the array, per device

// In host code `lf_static_scratch` is only a handle for the runtime, not an address a kernel
// could use; the device address has to be asked for, once per device, with that device current.
int static_scratch_for_current_device(float** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return LF_ECUDA;
    if (dev < 0 || dev >= LF_STATIC_MAX_DEVICES) return LF_ERESOURCE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_addr[dev]) {
        float* p = nullptr;
        // With CUDA's lazy module loading this look-up is also what loads the module that holds the
        // array and the kernel on this device: that reserves the array's megabyte and the code, and
        // it fails with an out-of-memory error if the process has already given all memory away.
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), lf_static_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? LF_ENOMEM : LF_ECUDA;
        }
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return LF_OK;
}

}  // namespace

extern "C" int lf_delta_step_static(const float* w_up, const float* delta_up, const float* a_l,
                                    float* delta_l, int N, void* cuda_stream)
{
    if (!w_up || !delta_up || !a_l || !delta_l) return LF_ENULL;
    const void* ps[] = {w_up, delta_up, a_l, delta_l};
    for (const void* p : ps)
        if (reinterpret_cast<uintptr_t>(p) & 15u) return LF_EALIGN;
    if (N < 1 || (N & 3) != 0) return LF_EINVAL;
    if (N > LF_STATIC_MAX_N) return LF_ECAPACITY;
    const int rows = dmv_rows_per_chunk(N);
    const int chunks = (N + rows - 1) / rows;
    const int strips = ((N >> 2) + DMV_STRIP4 - 1) / DMV_STRIP4;
    if (chunks > LF_STATIC_MAX_CHUNKS || strips > LF_STATIC_COUNTER_WORDS) return LF_ECAPACITY;

    float* scratch = nullptr;
    int rc = static_scratch_for_current_device(&scratch);
    if (rc != LF_OK) return rc;
    float* partial = scratch;
    unsigned* counters = reinterpret_cast<unsigned*>(scratch + LF_STATIC_PARTIAL_WORDS);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left.  The partial sums are fully rewritten
    // before they are read; the arrival counters must start at zero.
    if (cudaMemsetAsync(counters, 0, LF_STATIC_COUNTER_WORDS * sizeof(unsigned), s) != cudaSuccess)
        return LF_ECUDA;
    dim3 grid(strips, chunks);
    k_delta_matvec<<<grid, DMV_WARPS * 32, 0, s>>>(w_up, delta_up, a_l, delta_l, nullptr, partial,
                                                  counters, N, N, rows, chunks, LF_ACT_SIGMOID);
    return cudaGetLastError() == cudaSuccess ? LF_OK : LF_ECUDA;
}
