// Stand-alone timing probe (not part of libleapfrog): what one delta hand-off through L2 costs on
// this GPU.  The single-launch backward kernels publish delta^l as 8-byte {value, epoch} slots and
// every CTA polls them; the numbers below bound that step from underneath.
//   1. latency of one dependent slot load from L2, per multiprocessor (best and worst of 256 lines)
//   2. one poll round: a CTA of 256 threads reads N slots (everything already there), alone and
//      with 16 / 64 / 128 CTAs doing the same at the same time
//   3. the same poll round while gradient-sized store streams run: from four other warps of the
//      same CTA (32 KiB per round), from the 20 multiprocessors that do not poll, or both
// All loads and stores stay inside buffers allocated here; every loop is bounded.
// Build and run:  python -m paper_1801_04928_b200.handoff_probe
#include <cstdio>
#include <cuda_runtime.h>
#include <cooperative_groups.h>
namespace cg = cooperative_groups;

__device__ __forceinline__ unsigned long long ld_slot(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__global__ void k_latency(const unsigned long long* buf, int n_lines, int stride_words, unsigned* out)
{
    if (threadIdx.x != 0) return;
    for (int i = 0; i < n_lines; ++i) {
        const unsigned long long* p = buf + (size_t)i * stride_words;
        unsigned best = 0xffffffffu;
        for (int rep = 0; rep < 6; ++rep) {
            const long long t0 = clock64();
            const unsigned long long* q = p;
            unsigned long long v = 0;
#pragma unroll 1
            for (int k = 0; k < 4; ++k) {     // four dependent loads of the same line (contents: 0)
                v = ld_slot(q);
                q = p + v;
            }
            if (v == 0xdeadbeefULL) { out[0] = 1; return; }   // a real dependence before the clock is read
            const unsigned d = (unsigned)((clock64() - t0) / 4);
            if (rep > 0 && d < best) best = d;
        }
        out[(size_t)blockIdx.x * n_lines + i] = best;
    }
}

// threads 0..255 poll N slots; threads 256..383 stream stores.  CTAs >= pollers only store.
__global__ void k_poll(const unsigned long long* slots, int N, int pollers, int same_sm_store, int remote_store,
                       float* sink, size_t sink_floats_per_cta, unsigned* out)
{
    cg::grid_group g = cg::this_grid();
    const int tid = threadIdx.x;
    const bool poll_cta = (int)blockIdx.x < pollers;
    unsigned best = 0xffffffffu, sum = 0;
    float4* my = reinterpret_cast<float4*>(sink + (size_t)blockIdx.x * sink_floats_per_cta);
    for (int rep = 0; rep < 10; ++rep) {
        g.sync();
        if (tid < 256 && poll_cta) {
            const long long t0 = clock64();
            unsigned long long acc = 0;
            for (int i = tid; i < N; i += 256) acc += ld_slot(slots + i);
            if (acc == 0xdeadbeefULL) out[0] = 1;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            const unsigned d = (unsigned)(clock64() - t0);
            if (rep > 1) { if (d < best) best = d; sum += d; }
        } else if (tid >= 256 && ((poll_cta && same_sm_store) || (!poll_cta && remote_store))) {
            const int st = tid - 256;
            const int n4 = (poll_cta ? 32 : 256) * 1024 / 16;   // 32 KiB next to a poller, 256 KiB elsewhere
            for (int i = st; i < n4; i += 128) __stcs(my + i + (size_t)(rep & 3) * n4, make_float4(1.f, 2.f, 3.f, 4.f));
        }
    }
    if (tid == 0 && poll_cta) { out[2 * blockIdx.x] = best; out[2 * blockIdx.x + 1] = sum / 8; }
}

#define CHECK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e_), __FILE__, __LINE__); return 1; } } while (0)

int main()
{
    int nsm = 0;
    CHECK(cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, 0));
    // ---- 1. latency of one slot load
    {
        const int n_lines = 256, stride_words = 16 * 33;   // 128-byte lines, 4224 bytes apart
        unsigned long long* buf; unsigned* out;
        CHECK(cudaMalloc(&buf, (size_t)n_lines * stride_words * 8));
        CHECK(cudaMemset(buf, 0, (size_t)n_lines * stride_words * 8));
        CHECK(cudaMalloc(&out, (size_t)nsm * n_lines * 4));
        CHECK(cudaFuncSetAttribute(k_latency, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        k_latency<<<nsm, 32, 200 * 1024>>>(buf, n_lines, stride_words, out);   // one CTA per multiprocessor
        CHECK(cudaDeviceSynchronize());
        unsigned* h = new unsigned[(size_t)nsm * n_lines];
        CHECK(cudaMemcpy(h, out, (size_t)nsm * n_lines * 4, cudaMemcpyDeviceToHost));
        unsigned lo = ~0u, hi = 0; double sum = 0;
        for (size_t i = 0; i < (size_t)nsm * n_lines; ++i) { lo = h[i] < lo ? h[i] : lo; hi = h[i] > hi ? h[i] : hi; sum += h[i]; }
        printf("1. one dependent slot load from L2 (ld.relaxed.gpu.u64), %d multiprocessors x %d lines: "
               "best %u, mean %.0f, worst %u SM cycles\n", nsm, n_lines, lo, sum / ((double)nsm * n_lines), hi);
        delete[] h; cudaFree(buf); cudaFree(out);
    }
    // ---- 2. and 3. poll rounds
    const int grid = nsm < 148 ? nsm : 148;
    unsigned long long* slots; unsigned* out; float* sink;
    size_t per_cta = (size_t)4 * 256 * 1024 / 4;   // floats: four rounds of 256 KiB
    CHECK(cudaMalloc(&slots, 4096 * 8)); CHECK(cudaMemset(slots, 0, 4096 * 8));
    CHECK(cudaMalloc(&out, 2 * grid * 4)); CHECK(cudaMalloc(&sink, per_cta * 4 * grid));
    unsigned h[2 * 148];
    auto run = [&](int N, int pollers, int same, int remote, double* best, double* mean, unsigned* worst) -> int {
        void* args[] = {&slots, &N, &pollers, &same, &remote, &sink, &per_cta, &out};
        CHECK(cudaLaunchCooperativeKernel((void*)k_poll, dim3(grid), dim3(384), args, 0, 0));
        CHECK(cudaDeviceSynchronize());
        CHECK(cudaMemcpy(h, out, 2 * grid * 4, cudaMemcpyDeviceToHost));
        *best = 0; *mean = 0; *worst = 0;
        for (int i = 0; i < pollers; ++i) { *best += h[2 * i]; *mean += h[2 * i + 1]; *worst = h[2 * i + 1] > *worst ? h[2 * i + 1] : *worst; }
        *best /= pollers; *mean /= pollers;
        return 0;
    };
    double b, m; unsigned w;
    printf("2. one poll round of N slots by a CTA of 256 threads, everything already published (SM cycles: best / mean / worst CTA's mean)\n");
    for (int N : {256, 1024, 4096})
        for (int pollers : {1, 16, 64, 128}) {
            if (pollers > grid) continue;
            if (run(N, pollers, 0, 0, &b, &m, &w)) return 1;
            printf("   N %4d, %3d CTAs polling at once: %.0f / %.0f / %u\n", N, pollers, b, m, w);
        }
    printf("3. the same with store streams running (128 polling CTAs; the other %d multiprocessors store 256 KiB per round)\n", grid - 128);
    if (grid > 128)
        for (int N : {256, 1024})
            for (int same : {0, 1})
                for (int remote : {0, 1}) {
                    if (run(N, 128, same, remote, &b, &m, &w)) return 1;
                    printf("   N %4d, stores from the same CTA's other warps: %s, from the other multiprocessors: %s: %.0f / %.0f / %u\n",
                           N, same ? "yes" : "no ", remote ? "yes" : "no ", b, m, w);
                }
    return 0;
}
