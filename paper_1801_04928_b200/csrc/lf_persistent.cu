// Persistent single-launch backward pass for one sample (B = 1): Eq. bp1, the Eq. bp2 chain and
// Eq. bp3/bp4 of every layer in ONE kernel.
//
// Roles.  The grid is a row of thread-block clusters of 8 CTAs.
//   * Chain clusters.  Cluster q owns the column strip [q*Ws, (q+1)*Ws) of every weight matrix;
//     inside it CTA c owns the rows [c*Hr, (c+1)*Hr).  For layer step s (reading w^s, producing
//     delta^{s-1}) a CTA multiplies its tile by delta^s of its rows, the 8 CTAs of the cluster
//     add their partial column sums through distributed shared memory (each CTA finishes 1/8 of
//     the strip), apply sigma' and publish delta^{s-1}.  Weight tiles do not depend on delta, so
//     they are fetched by TMA several sub-tiles (and layers) ahead of the chain.
//   * Fused variant: the pass over a tile of w^s also stores the same tile of gw^s =
//     delta^s (x) a^{s-1} (both already known); gw^1 is stored by a tail pass.
//   * Leapfrog variant: extra worker clusters are split into k groups; group (L-l) mod k waits
//     for delta^l and streams gw^l out (Section 3: each worker handles every k-th layer).  The
//     chain CTAs then only read.
//
// delta crosses CTAs through an exchange buffer of 8-byte slots {value, epoch}: one 64-bit store
// publishes a value together with its "ready" tag, one 64-bit load polls both, so no fence and no
// separate flag is needed.  The epoch changes with every call, so the buffer is never cleared.
// Every wait (slot poll, TMA barrier) is bounded by a time budget; on expiry the CTA raises the
// status word, stops waiting for the rest of the launch and runs to completion with whatever it
// has, so cluster barriers still see every thread and the kernel always ends.
#include <cuda.h>

#include "lf_internal.h"

namespace {

constexpr int PK_THREADS = 256;
constexpr int PK_CLUSTER = 8;
constexpr int PK_STAGE_FLOATS = 8192;  // 32 KiB per pipeline stage
constexpr int PK_STAGES = 6;
constexpr int PK_MAX_NCB = 4;          // column blocks per strip (strip width <= 4 * 256)
constexpr int PK_MAX_SLICE = 128;      // strip columns finished per CTA (strip / 8)

struct PkParams {
    int L, N;
    int Qc;        // chain clusters
    int Qw;        // worker clusters (0 in the fused variant)
    int fused;     // 1: chain CTAs store gw tiles
    int Wc;        // columns per column block (32, 64, 128 or 256)
    int nCB;       // column blocks per strip
    int Ws;        // strip width = Wc * nCB
    int Hr;        // rows per chain CTA
    int R;         // rows per sub-tile = PK_STAGE_FLOATS / Wc
    int nRB;       // row blocks per layer
    int slice;     // Ws / 8
    int keff;      // effective leapfrog workers
    unsigned epoch;
    unsigned long long budget_ns;
    const float* a;
    const float* y;
    float* delta;
    float* gw;
    float* gb;
    unsigned long long* xch;  // [L][N] slots
    unsigned* status;
};

// ---- small PTX wrappers ----------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p)
{
    return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void tma_load_3d(unsigned dst, const CUtensorMap* map, unsigned bar,
                                            int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;"
                 ::: "memory");
}
__device__ __forceinline__ unsigned cluster_ctarank()
{
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ unsigned map_to_cta(unsigned local_addr, unsigned rank)
{
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(unsigned addr, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_slot(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_slot(unsigned long long* p, float value, unsigned epoch)
{
    unsigned long long v = ((unsigned long long)epoch << 32) | (unsigned long long)__float_as_uint(value);
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_stream4(float* p, float4 v)
{
    __stcs(reinterpret_cast<float4*>(p), v);
}

struct PkShared {
    unsigned long long full[PK_STAGES];  // TMA arrival barriers
    volatile unsigned abort_flag;        // set once a wait of this CTA has run out
};

// Wait until slot *p carries this call's epoch; returns the value (0 after a timeout).
__device__ __forceinline__ float wait_slot(const unsigned long long* p, const PkParams& P,
                                           PkShared* sh)
{
    unsigned long long v = ld_slot(p);
    if ((unsigned)(v >> 32) == P.epoch) return __uint_as_float((unsigned)v);
    if (sh->abort_flag) return 0.f;
    const unsigned long long t0 = globaltimer_ns();
    unsigned spins = 0;
    for (;;) {
        v = ld_slot(p);
        if ((unsigned)(v >> 32) == P.epoch) return __uint_as_float((unsigned)v);
        if ((++spins & 31u) == 0u) {
            if (sh->abort_flag) return 0.f;
            if (globaltimer_ns() - t0 > P.budget_ns || (((spins & 1023u) == 0u) && *((volatile unsigned*)P.status) != 0u)) {
                atomicOr(P.status, LF_DEV_TIMEOUT_FLAG);
                sh->abort_flag = 1u;
                return 0.f;
            }
        }
    }
}

__device__ __forceinline__ void wait_full(unsigned bar, unsigned parity, const PkParams& P,
                                          PkShared* sh)
{
    if (mbar_try_wait(bar, parity)) return;
    if (sh->abort_flag) return;
    const unsigned long long t0 = globaltimer_ns();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 15u) == 0u) {
            if (sh->abort_flag) return;
            if (globaltimer_ns() - t0 > P.budget_ns) {
                atomicOr(P.status, LF_DEV_TIMEOUT_BARRIER);
                sh->abort_flag = 1u;
                return;
            }
        }
    }
}

// Eq. bp4 for the rows [row0, row1) and all N columns: the leapfrog worker's store stream.
__device__ void worker_store_rows(const PkParams& P, int l, int row0, int row1, float* d_rows,
                                  float* a_sm, PkShared* sh)
{
    const int N = P.N, n4 = N >> 2;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const float* a_prev = P.a + (size_t)(l - 1) * N;
    for (int c = tid; c < n4; c += PK_THREADS)
        reinterpret_cast<float4*>(a_sm)[c] = reinterpret_cast<const float4*>(a_prev)[c];
    const unsigned long long* slots = P.xch + (size_t)(l - 1) * N;
    for (int r = row0 + tid; r < row1; r += PK_THREADS) d_rows[r - row0] = wait_slot(slots + r, P, sh);
    __syncthreads();
    float* gw_l = P.gw + (size_t)(l - 1) * N * N;
    for (int r = row0 + warp; r < row1; r += PK_THREADS / 32) {
        const float d = d_rows[r - row0];
        float* out = gw_l + (size_t)r * N;
        for (int c = lane; c < n4; c += 32) {
            float4 a4 = reinterpret_cast<const float4*>(a_sm)[c];
            st_stream4(out + 4 * c, make_float4(d * a4.x, d * a4.y, d * a4.z, d * a4.w));
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(PK_THREADS, 1)
k_backward_persistent(const __grid_constant__ CUtensorMap w_map, const PkParams P)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    float* stages = reinterpret_cast<float*>(smem_raw);                       // PK_STAGES x 32 KiB
    float* d_rows = stages + PK_STAGES * PK_STAGE_FLOATS;                     // nRB*R (<= 2304)
    float* red = d_rows + 2304;                                               // 256 float4
    float* recv = red + PK_THREADS * 4;                                       // [2][8][PK_MAX_SLICE]
    PkShared* sh = reinterpret_cast<PkShared*>(recv + 2 * PK_CLUSTER * PK_MAX_SLICE);

    const int tid = threadIdx.x;
    const int N = P.N, L = P.L;
    const int cluster_id = blockIdx.x / PK_CLUSTER;
    const int c = (int)cluster_ctarank();

    if (tid == 0) {
        for (int i = 0; i < PK_STAGES; ++i) mbar_init(smem_u32(&sh->full[i]), 1);
        sh->abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // ===================== leapfrog worker clusters ==========================================
    if (cluster_id >= P.Qc) {
        const int Wn = P.Qw * PK_CLUSTER;
        const int wi = (cluster_id - P.Qc) * PK_CLUSTER + c;
        const int G = P.keff < Wn ? P.keff : Wn;     // groups that really exist
        const int g = wi % G, m = wi / G;
        const int Mg = (Wn - g + G - 1) / G;          // members of my group
        const int rpm = (N + Mg - 1) / Mg;            // rows per member
        const int row0 = m * rpm, row1 = min(N, row0 + rpm);
        float* a_sm = stages;                         // N floats (N <= 16384 fits one... two stages)
        float* dr = stages + 16384;                   // up to N floats
        for (int l = L; l >= 1; --l) {
            if ((((L - l) % P.keff) % G) != g) continue;   // not a layer of my group
            if (row0 < row1) worker_store_rows(P, l, row0, row1, dr, a_sm, sh);
        }
        cluster_sync_all();   // matched by nothing else: keeps the cluster's CTAs exiting together
        return;
    }

    // ===================== chain clusters ====================================================
    const int q = cluster_id;
    const int Wc = P.Wc, nCB = P.nCB, R = P.R, nRB = P.nRB, Hr = P.Hr, Ws = P.Ws;
    const int WC4 = Wc >> 2;
    const int RG = PK_THREADS / WC4;       // row groups
    const int tcol = tid % WC4, trow = tid / WC4;
    const int row_base = c * Hr;
    const int row_end = min(N, row_base + Hr);
    const int col_base = q * Ws;
    const int nSub = nCB * nRB;
    const int total = (L - 1) * nSub;
    const unsigned stage_bytes = (unsigned)(R * Wc * sizeof(float));
    const int Hr_pad = nRB * R;

    // producer: issue the TMA load of sub-tile `it` of this CTA's sequence
    auto issue = [&](int it) {
        const int step = it / nSub, sub = it - step * nSub;
        const int s = L - step;                 // w^s
        const int cb = sub / nRB, rb = sub - cb * nRB;
        const int st = it % PK_STAGES;
        const unsigned bar = smem_u32(&sh->full[st]);
        mbar_expect_tx(bar, stage_bytes);
        tma_load_3d(smem_u32(stages + (size_t)st * PK_STAGE_FLOATS), &w_map, bar,
                    col_base + cb * Wc, row_base + rb * R, s - 1);
    };
    if (tid == 0) {
        const int pre = total < PK_STAGES ? total : PK_STAGES;
        for (int it = 0; it < pre; ++it) issue(it);
    }

    // ---- Eq. bp1: delta^L for my rows (every cluster computes it for itself)
    {
        const float* aL = P.a + (size_t)L * N;
        for (int r = tid; r < Hr_pad; r += PK_THREADS) {
            const int row = row_base + r;
            float d = 0.f;
            if (r < Hr && row < N) {
                const float av = aL[row];
                d = (av - P.y[row]) * (av * (1.0f - av));
                if (q == 0) {
                    P.delta[(size_t)(L - 1) * N + row] = d;
                    P.gb[(size_t)(L - 1) * N + row] = d;                  // Eq. bp3
                    if (P.Qw > 0) st_slot(P.xch + (size_t)(L - 1) * N + row, d, P.epoch);
                }
            }
            d_rows[r] = d;
        }
    }
    __syncthreads();

    int it = 0;
    for (int s = L; s >= 2; --s) {
        // a^{s-1}: columns of my strip (for the gw^s tile) and of my slice (for sigma')
        const float* a_prev = P.a + (size_t)(s - 1) * N;
        float4 a4[PK_MAX_NCB];
#pragma unroll
        for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
            a4[cb] = make_float4(0.f, 0.f, 0.f, 0.f);
            const int col = col_base + cb * Wc + tcol * 4;
            if (cb < nCB && P.fused && col < N) a4[cb] = *reinterpret_cast<const float4*>(a_prev + col);
        }
        const int my_col = col_base + c * P.slice + tid;   // the column this thread finishes (tid < slice)
        float a_mine = 0.f;
        if (tid < P.slice && my_col < N) a_mine = a_prev[my_col];

        float* gw_s = P.gw + (size_t)(s - 1) * N * N;
        const int par = s & 1;
        float* recv_p = recv + par * PK_CLUSTER * PK_MAX_SLICE;

#pragma unroll
        for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
            if (cb >= nCB) break;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            const int col = col_base + cb * Wc + tcol * 4;
            const bool col_ok = col < N;
            for (int rb = 0; rb < nRB; ++rb, ++it) {
                const int st = it % PK_STAGES;
                wait_full(smem_u32(&sh->full[st]), (unsigned)((it / PK_STAGES) & 1), P, sh);
                const float4* tile = reinterpret_cast<const float4*>(stages + (size_t)st * PK_STAGE_FLOATS);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = trow + i * RG;            // row inside the sub-tile
                    const float4 wv = tile[r * WC4 + tcol];
                    const int rr = rb * R + r;              // row inside my chunk
                    const float d = d_rows[rr];
                    acc.x = fmaf(wv.x, d, acc.x);
                    acc.y = fmaf(wv.y, d, acc.y);
                    acc.z = fmaf(wv.z, d, acc.z);
                    acc.w = fmaf(wv.w, d, acc.w);
                    if (P.fused) {
                        const int row = row_base + rr;
                        if (col_ok && rr < Hr && row < row_end)
                            st_stream4(gw_s + (size_t)row * N + col,
                                       make_float4(d * a4[cb].x, d * a4[cb].y, d * a4[cb].z, d * a4[cb].w));
                    }
                }
                __syncthreads();   // every thread is done with this stage
                if (tid == 0 && it + PK_STAGES < total && !sh->abort_flag) issue(it + PK_STAGES);
            }
            // partial column sums of this column block: add the RG row groups in order
            reinterpret_cast<float4*>(red)[tid] = acc;
            __syncthreads();
            if (tid < WC4) {
                float4 sum = reinterpret_cast<const float4*>(red)[tid];
                for (int gidx = 1; gidx < RG; ++gidx) {
                    const float4 t = reinterpret_cast<const float4*>(red)[gidx * WC4 + tid];
                    sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
                }
                // hand the four columns to the CTA that finishes them
                const int cs = cb * Wc + tid * 4;            // column inside the strip
                const int owner = cs / P.slice, off = cs - owner * P.slice;
                const unsigned base = map_to_cta(smem_u32(recv_p + c * PK_MAX_SLICE + off), (unsigned)owner);
                st_cluster_f32(base + 0, sum.x);
                st_cluster_f32(base + 4, sum.y);
                st_cluster_f32(base + 8, sum.z);
                st_cluster_f32(base + 12, sum.w);
            }
            __syncthreads();
        }
        cluster_sync_all();   // all partial sums of the strip have landed
        if (tid < P.slice) {
            float v = recv_p[tid];
#pragma unroll
            for (int cc = 1; cc < PK_CLUSTER; ++cc) v += recv_p[cc * PK_MAX_SLICE + tid];
            if (my_col < N) {
                const float d = v * (a_mine * (1.0f - a_mine));   // Eq. bp2
                st_slot(P.xch + (size_t)(s - 2) * N + my_col, d, P.epoch);
                P.delta[(size_t)(s - 2) * N + my_col] = d;
                P.gb[(size_t)(s - 2) * N + my_col] = d;           // Eq. bp3
            }
        }
        // delta^{s-1} of my rows, from whichever clusters finished those columns
        {
            const unsigned long long* slots = P.xch + (size_t)(s - 2) * N;
            for (int r = tid; r < Hr_pad; r += PK_THREADS) {
                const int row = row_base + r;
                float d = 0.f;
                if (r < Hr && row < N) d = wait_slot(slots + row, P, sh);
                d_rows[r] = d;
            }
        }
        __syncthreads();
    }

    // ---- tail: gw^1 = delta^1 (x) a^0 for my tile (fused variant)
    if (P.fused) {
        const float* a0 = P.a;
#pragma unroll
        for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
            if (cb >= nCB) break;
            const int col = col_base + cb * Wc + tcol * 4;
            if (col >= N) continue;
            const float4 av = *reinterpret_cast<const float4*>(a0 + col);
            for (int rr = trow; rr < Hr; rr += RG) {
                const int row = row_base + rr;
                if (row >= row_end) break;
                const float d = d_rows[rr];
                st_stream4(P.gw + (size_t)row * N + col, make_float4(d * av.x, d * av.y, d * av.z, d * av.w));
            }
        }
    }
    cluster_sync_all();   // no CTA leaves while a peer may still address its shared memory
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                    const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                    const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_fn()
{
    static encode_tiled_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

constexpr size_t PK_SMEM_BYTES = (size_t)PK_STAGES * PK_STAGE_FLOATS * 4 + 2304 * 4 + PK_THREADS * 16 +
                                 2 * PK_CLUSTER * PK_MAX_SLICE * 4 + 128;

struct PkPlan {
    bool ok;
    int Qmax, Qc, Qw, Wc, nCB, Ws, Hr, R, nRB, slice;
};

int max_active_clusters(const lf_ctx* c)
{
    static int cached_dev = -1, cached = 0;
    if (cached_dev == c->device) return cached;
    if (cudaFuncSetAttribute(k_backward_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)PK_SMEM_BYTES) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(PK_CLUSTER * 16);
    cfg.blockDim = dim3(PK_THREADS);
    cfg.dynamicSmemBytes = PK_SMEM_BYTES;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = PK_CLUSTER; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_backward_persistent, &cfg) != cudaSuccess) {
        cudaGetLastError();
        n = 0;
    }
    cached_dev = c->device;
    cached = n;
    return n;
}

PkPlan make_plan(const lf_ctx* c, int variant)
{
    PkPlan p = {};
    if (c->B != 1) return p;
    if ((size_t)c->smem_optin < PK_SMEM_BYTES) return p;
    if (!get_encode_fn()) return p;
    p.Qmax = max_active_clusters(c);
    if (p.Qmax > 18) p.Qmax = 18;
    int Qc_budget = p.Qmax;
    if (variant == LF_VARIANT_PERSISTENT) {
        if (p.Qmax < 2) return p;
        Qc_budget = p.Qmax / 2;
    }
    if (Qc_budget < 1) return p;
    const int N = c->N;
    int need = (N + Qc_budget - 1) / Qc_budget;      // strip width needed
    int Wc = 32;
    while (Wc < need && Wc < 256) Wc <<= 1;
    int nCB = 1;
    while (Wc * nCB < need) nCB <<= 1;
    if (nCB > PK_MAX_NCB) return p;
    p.Wc = Wc; p.nCB = nCB; p.Ws = Wc * nCB;
    p.Qc = (N + p.Ws - 1) / p.Ws;
    p.Qw = variant == LF_VARIANT_PERSISTENT ? p.Qmax - p.Qc : 0;
    p.R = PK_STAGE_FLOATS / Wc;
    p.Hr = (N + PK_CLUSTER - 1) / PK_CLUSTER;
    p.nRB = (p.Hr + p.R - 1) / p.R;
    p.slice = p.Ws / PK_CLUSTER;
    if (p.slice > PK_MAX_SLICE || p.nRB * p.R > 2304) return p;
    if (variant == LF_VARIANT_PERSISTENT && N > 16384) return p;
    p.ok = true;
    return p;
}

}  // namespace

size_t lf_sync_words_needed(const lf_ctx* c)
{
    // exchange slots: L * N 64-bit words (only single-sample contexts use them)
    if (c->B != 1) return 64;
    return (size_t)2 * c->L * c->N + 64;
}

bool lf_persistent_supported(const lf_ctx* c, int variant)
{
    if (variant != LF_VARIANT_PERSISTENT && variant != LF_VARIANT_FUSED) return false;
    return make_plan(c, variant).ok;
}

int lf_auto_variant(const lf_ctx* c)
{
    if (c->B != 1) return LF_VARIANT_STREAMS;
    return make_plan(c, LF_VARIANT_FUSED).ok ? LF_VARIANT_FUSED : LF_VARIANT_STREAMS;
}

int lf_backward_persistent(lf_ctx* c, int variant, const float* w, const float* z, const float* a,
                           const float* y, float* delta, float* gw, float* gb)
{
    (void)z;
    PkPlan pl = make_plan(c, variant);
    if (!pl.ok) return LF_ERESOURCE;
    // tensor map over w as [L][N][N], box = Wc columns x R rows x 1 layer
    if (!c->w_map_valid || c->w_map_ptr != w || c->w_map_wc != pl.Wc) {
        CUtensorMap* m = reinterpret_cast<CUtensorMap*>(c->w_map_storage);
        cuuint64_t dims[3] = {(cuuint64_t)c->N, (cuuint64_t)c->N, (cuuint64_t)c->L};
        cuuint64_t strides[2] = {(cuuint64_t)c->N * 4, (cuuint64_t)c->N * c->N * 4};
        cuuint32_t box[3] = {(cuuint32_t)pl.Wc, (cuuint32_t)pl.R, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = get_encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(w), dims,
                                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                     CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            c->last_cuda_error = (int)r;
            return LF_ECUDA;
        }
        c->w_map_valid = true; c->w_map_ptr = w; c->w_map_wc = pl.Wc;
    }
    c->epoch += 1;
    if (c->epoch == 0) c->epoch = 1;

    PkParams P = {};
    P.L = c->L; P.N = c->N; P.Qc = pl.Qc; P.Qw = pl.Qw;
    P.fused = variant == LF_VARIANT_FUSED ? 1 : 0;
    P.Wc = pl.Wc; P.nCB = pl.nCB; P.Ws = pl.Ws; P.Hr = pl.Hr; P.R = pl.R; P.nRB = pl.nRB;
    P.slice = pl.slice; P.keff = c->keff; P.epoch = c->epoch;
    P.budget_ns = (unsigned long long)c->wait_budget_us * 1000ull;
    P.a = a; P.y = y; P.delta = delta; P.gw = gw; P.gb = gb;
    P.xch = reinterpret_cast<unsigned long long*>(c->sync_words);
    P.status = c->status_dev;

    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)PK_SMEM_BYTES));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((pl.Qc + pl.Qw) * PK_CLUSTER);
    cfg.blockDim = dim3(PK_THREADS);
    cfg.dynamicSmemBytes = PK_SMEM_BYTES;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = PK_CLUSTER; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const CUtensorMap* mp = reinterpret_cast<const CUtensorMap*>(c->w_map_storage);
    LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_persistent, *mp, P));
    c->stats.launches_backward = 1;
    c->stats.chain_ctas = pl.Qc * PK_CLUSTER;
    c->stats.worker_ctas = pl.Qw * PK_CLUSTER;
    return LF_OK;
}

void lf_persistent_release(lf_ctx*) {}
