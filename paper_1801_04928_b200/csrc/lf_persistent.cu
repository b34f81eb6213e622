// Persistent single-launch backward pass for one sample (B = 1): Eq. bp1, the Eq. bp2 chain and
// Eq. bp3/bp4 of every layer in ONE kernel.
//
// Grid.  A row of thread-block clusters of C CTAs (C = 2, 4 or 8: whichever puts the most SMs
// to work), one CTA per SM, 256 threads per CTA.
//   * Chain clusters.  Cluster q owns the column strip [q*Ws, (q+1)*Ws) of every weight matrix;
//     inside it CTA c owns the rows [c*Hr, (c+1)*Hr).  For layer step s (reading w^s, producing
//     delta^{s-1}) the CHAIN WARPS (0-3) of a CTA multiply its tile by delta^s of its rows, send
//     their partial column sums through distributed shared memory to the CTA of the cluster that
//     finishes those columns (each CTA finishes 1/C of the strip), which adds them, applies
//     sigma' and publishes delta^{s-1}.  Weight tiles do not depend on delta, so they are
//     fetched by TMA several sub-tiles (and layers) ahead of the chain.
//   * Fused variant: the STORE WARPS (4-7) of the same CTA stream the tile of gw^s =
//     delta^s (x) a^{s-1} out while the chain warps go on; gw^1 follows after the last step.
//   * Leapfrog variant: extra worker clusters are split into k groups; group (L-l) mod k waits
//     for delta^l and streams gw^l out (Section 3: each worker handles every k-th layer).  The
//     chain CTAs then only read.
//
// Hand-offs.  delta crosses clusters through an exchange buffer of 8-byte slots {value, epoch}:
// one 64-bit store publishes a value together with its "ready" tag and one 64-bit load polls
// both, so no fence and no separate flag is needed; the epoch changes with every call, so the
// buffer is never cleared.  Partial sums cross CTAs of a cluster by st.async, which writes the
// data and credits its bytes to an mbarrier of the receiving CTA; chain and store warps of a CTA hand the delta buffers back and
// forth through two pairs of mbarriers.  Every wait is bounded by a time budget; on expiry the
// CTA raises the status word, stops waiting for the rest of the launch and runs to the end with
// whatever it has, so the kernel always terminates.
#include <cuda.h>

#include "lf_internal.h"
#include "lf_ptx.cuh"

namespace {

constexpr int PK_THREADS = 256;          // chain warps 0-3 and store warps 4-7
constexpr int PK_LAUNCH_THREADS = 288;   // + warp 8, whose lane 0 is the TMA producer of a chain CTA
constexpr int PK_PRODUCER_WARP = 8;
constexpr int PK_CHAIN_THREADS = 128;   // warps 0-3
constexpr int PK_CHAIN_WARPS = 4;
constexpr int PK_MAX_CLUSTER = 8;       // cluster sizes 2, 4 and 8 are used
constexpr int PK_STAGE_FLOATS = 8192;   // 32 KiB per pipeline stage
constexpr int PK_STAGES = 6;
constexpr int PK_MAX_NCB = 4;           // column blocks per strip (strip width <= 4 * 256)
constexpr int PK_MAX_SLICE = 128;       // strip columns finished per CTA (strip / C)
constexpr int PK_SGD_BATCH = 16;        // fused weight update: loads of w a thread keeps in flight
constexpr int PK_DROWS = 2176;          // floats of delta held per CTA and buffer (tile rows, padded)

struct PkParams {
    int L, N;
    int C;         // CTAs per cluster
    int Qc;        // chain clusters
    int Qw;        // worker clusters (0 in the fused variant)
    int shard_rank, shard_count;   // the workers store layer l only if (L - l) % shard_count == shard_rank
    int top_given;     // 1: delta of the top layer is already in `delta` (the launch covers a run of layers
                       //    below the network's own top layer); 0: Eq. bp1 is computed here
    int depth_shift;   // layers between the run's top layer and the network's: added to (L - l) wherever
                       //    a layer is given to a shard or a worker group
    int fused;     // 1: chain CTAs store gw tiles
    int Wc;        // columns per column block (32, 64, 128 or 256)
    int nCB;       // column blocks per strip
    int Ws;        // strip width = Wc * nCB
    int Hr;        // rows per chain CTA
    int R;         // rows per sub-tile = PK_STAGE_FLOATS / Wc
    int nRB;       // row blocks per layer
    int slice;     // Ws / C
    int keff;      // effective leapfrog workers
    int withhold;  // test hook: chain CTA 0 publishes nothing (the others' waits must expire)
    int cost;      // enum lf_cost: which grad_a C enters Eq. bp1
    int act;       // enum lf_activation: sigma' from the stored activations
    unsigned epoch;
    unsigned long long budget_ns;
    const float* a;
    const float* y;
    const float* w_sub;       // fused weight update: store w_sub - eta * gw in place of gw (null: plain gw)
    float eta;
    float* delta;
    float* gw;
    float* gb;
    unsigned long long* xch;  // [L][N] slots
    unsigned* status;
#ifdef LF_PK_TRACE
    unsigned long long* trace;  // [2 CTAs][L][16] SM-clock stamps (debug builds only)
#endif
};

// ---- PTX wrappers: the shared ones of lf_ptx.cuh, and two of this kernel's own -------------------
using namespace lfptx;
__device__ __forceinline__ void chain_sync()   // the four chain warps only
{
    asm volatile("bar.sync 1, 128;" ::: "memory");
}
// Store four floats into the shared memory of a CTA of the cluster and credit 16 bytes to an
// mbarrier there (both addresses from mapa): data and "it has arrived" travel together, no fence.
__device__ __forceinline__ void st_async_f32x4(unsigned cluster_addr, float4 v, unsigned cluster_bar)
{
    asm volatile(
        "st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
        ::"r"(cluster_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(cluster_bar)
        : "memory");
}

// Debug builds (-DLF_PK_TRACE) record SM-clock stamps of each chain step of two CTAs.
#ifdef LF_PK_TRACE
#define PK_STAMP(slot)                                                                       \
    do {                                                                                     \
        if (tid == 0 && (blockIdx.x == 0 || blockIdx.x == 77))                               \
            P.trace[((blockIdx.x == 0 ? 0 : 1) * (size_t)P.L + (size_t)(P.L - s)) * 16 + (slot)] = \
                (unsigned long long)clock64();                                               \
    } while (0)
#else
#define PK_STAMP(slot) do { } while (0)
#endif

struct PkShared {
    unsigned long long full[PK_STAGES];  // TMA arrival, one per stage
    unsigned long long part_ready[2];    // partial sums of a step have landed here (by step parity)
    unsigned long long d_ready[2];       // chain warps filled delta buffer p
    unsigned long long d_free[2];        // store warps are done with delta buffer p
    unsigned long long st_done[PK_STAGES];   // fused weight update: store warps have read the stage
    unsigned long long empty[PK_STAGES];     // the four chain warps have read the stage
    volatile unsigned abort_flag;        // set once a wait of this CTA has run out
};

__device__ __forceinline__ void raise_timeout(const PkParams& P, PkShared* sh, unsigned bit)
{
    atomicOr(P.status, bit);
    sh->abort_flag = 1u;
}

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
            if (globaltimer_ns() - t0 > P.budget_ns ||
                (((spins & 1023u) == 0u) && *((volatile unsigned*)P.status) != 0u)) {
                raise_timeout(P, sh, LF_DEV_TIMEOUT_FLAG);
                return 0.f;
            }
        }
    }
}

// Bounded wait on an mbarrier of this CTA (CLUSTER = arrivals come from other CTAs).
template <bool CLUSTER>
__device__ __forceinline__ void wait_bar(unsigned bar, unsigned parity, const PkParams& P,
                                         PkShared* sh)
{
    if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return;
    if (sh->abort_flag) return;
    const unsigned long long t0 = globaltimer_ns();
    unsigned spins = 0;
    while (!(CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity))) {
        if ((++spins & 15u) == 0u) {
            if (sh->abort_flag) return;
            if (globaltimer_ns() - t0 > P.budget_ns) {
                raise_timeout(P, sh, LF_DEV_TIMEOUT_BARRIER);
                return;
            }
        }
    }
}

// Eq. bp4 for the rows [row0, row1) and all N columns: the leapfrog worker's store stream.
template <bool UPDATE>
__device__ void worker_store_rows(const PkParams& P, int l, int row0, int row1, float* d_rows,
                                  float* a_sm, PkShared* sh)
{
    const int N = P.N, n4 = N >> 2;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const float* a_prev = P.a + (size_t)(l - 1) * N;
    if (tid < PK_THREADS) {   // (the ninth warp has no part in a worker CTA; it only keeps the barriers whole)
        for (int c = tid; c < n4; c += PK_THREADS)
            reinterpret_cast<float4*>(a_sm)[c] = reinterpret_cast<const float4*>(a_prev)[c];
        const unsigned long long* slots = P.xch + (size_t)(l - 1) * N;
        for (int r = row0 + tid; r < row1; r += PK_THREADS) d_rows[r - row0] = wait_slot(slots + r, P, sh);
    }
    __syncthreads();
    float* gw_l = P.gw + (size_t)(l - 1) * N * N;
    const float* w_l = UPDATE ? P.w_sub + (size_t)(l - 1) * N * N : nullptr;
    for (int r = row0 + warp; warp < PK_THREADS / 32 && r < row1; r += PK_THREADS / 32) {
        const float d = d_rows[r - row0];
        float* out = gw_l + (size_t)r * N;
        if (UPDATE) {
            const float4* w_row = reinterpret_cast<const float4*>(w_l + (size_t)r * N);
            for (int c0 = lane; c0 < n4; c0 += 32 * PK_SGD_BATCH) {
                float4 wv[PK_SGD_BATCH];
#pragma unroll
                for (int u = 0; u < PK_SGD_BATCH; ++u)
                    if (c0 + 32 * u < n4) wv[u] = __ldcg(w_row + c0 + 32 * u);
#pragma unroll
                for (int u = 0; u < PK_SGD_BATCH; ++u) {
                    const int c = c0 + 32 * u;
                    if (c < n4) {
                        const float4 a4 = reinterpret_cast<const float4*>(a_sm)[c];
                        st_stream4(out + 4 * c, lf_sgd_apply4(P.eta, wv[u], make_float4(d * a4.x, d * a4.y, d * a4.z, d * a4.w)));
                    }
                }
            }
        } else {
#pragma unroll 4
            for (int c = lane; c < n4; c += 32) {
                float4 a4 = reinterpret_cast<const float4*>(a_sm)[c];
                st_stream4(out + 4 * c, make_float4(d * a4.x, d * a4.y, d * a4.z, d * a4.w));
            }
        }
    }
    __syncthreads();
}

// Fused weight update of one column block of a CTA's tile (store warps of the fused variant):
// out[rr][0..3] = w_in[rr][0..3] - eta * d[rr] * av for this thread's rows rr = trow, trow + RG, ...
// A load costs a round trip that a store does not: every thread keeps PK_SGD_BATCH loads of w in
// flight (a rotating queue in registers: use the oldest, then reissue its slot) so that the reads
// keep up with the store stream.  Used for layer 1, which the chain never reads (the other layers
// take w from the chain's shared-memory stages).
// Not inlined: the queue would otherwise be live across the caller's unrolled column blocks.
__device__ __noinline__ void store_tile_updated(const float* __restrict__ w_in, float* __restrict__ out,
                                                const float* dr, float4 av, int rows, int trow, int RG, int N,
                                                float eta)
{
    const int n_mine = rows > trow ? (rows - trow + RG - 1) / RG : 0;   // rows of this thread
    float4 wq[PK_SGD_BATCH];
#pragma unroll
    for (int u = 0; u < PK_SGD_BATCH; ++u)
        if (u < n_mine) wq[u] = __ldcg(reinterpret_cast<const float4*>(w_in + (size_t)(trow + u * RG) * N));
    for (int base = 0; base < n_mine; base += PK_SGD_BATCH) {
#pragma unroll
        for (int u = 0; u < PK_SGD_BATCH; ++u) {
            const int idx = base + u;
            if (idx < n_mine) {
                const int rr = trow + idx * RG;
                const float d = dr[rr];
                st_stream4(out + (size_t)rr * N, lf_sgd_apply4(eta, wq[u], make_float4(d * av.x, d * av.y, d * av.z, d * av.w)));
                if (idx + PK_SGD_BATCH < n_mine)
                    wq[u] = __ldcg(reinterpret_cast<const float4*>(w_in + (size_t)(rr + PK_SGD_BATCH * RG) * N));
            }
        }
    }
}

// UPDATE = true: the instance behind lf_backward_sgd (P.w_sub set); the plain instance carries
// none of its code.
template <bool UPDATE>
__global__ void __launch_bounds__(PK_LAUNCH_THREADS, 1)
k_backward_persistent(const __grid_constant__ CUtensorMap w_map, const PkParams P)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    float* stages = reinterpret_cast<float*>(smem_raw);                       // PK_STAGES x 32 KiB
    float* d_rows = stages + PK_STAGES * PK_STAGE_FLOATS;                     // [2][PK_DROWS]
    float4* red = reinterpret_cast<float4*>(d_rows + 2 * PK_DROWS);           // [2][4 warps][32 lanes]
    float* recv = reinterpret_cast<float*>(red + 2 * PK_CHAIN_THREADS);       // [2][C][PK_MAX_SLICE]
    PkShared* sh = reinterpret_cast<PkShared*>(recv + 2 * PK_MAX_CLUSTER * PK_MAX_SLICE);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = P.N, L = P.L, C = P.C;
    const int cluster_id = blockIdx.x / C;
    const int c = (int)cluster_ctarank();
    const bool is_chain_cluster = cluster_id < P.Qc;

    if (tid == 0) {
        for (int i = 0; i < PK_STAGES; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->st_done[i]), PK_THREADS - PK_CHAIN_THREADS);
            mbar_init(smem_u32(&sh->empty[i]), PK_CHAIN_WARPS);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh->part_ready[i]), 1);
            mbar_init(smem_u32(&sh->d_ready[i]), PK_CHAIN_THREADS);
            mbar_init(smem_u32(&sh->d_free[i]), PK_THREADS - PK_CHAIN_THREADS);
        }
        sh->abort_flag = 0u;
        mbar_fence_init();
    }
    __syncthreads();
    cluster_sync_all();   // every CTA's barriers exist before a peer can arrive on them

    // ===================== leapfrog worker clusters ==========================================
    if (!is_chain_cluster) {
        const int Wn = P.Qw * C;
        const int wi = (cluster_id - P.Qc) * C + c;
        const int G = P.keff < Wn ? P.keff : Wn;     // groups that really exist
        const int g = wi % G, m = wi / G;
        const int Mg = (Wn - g + G - 1) / G;          // members of my group
        const int rpm = (N + Mg - 1) / Mg;            // rows per member
        const int row0 = m * rpm, row1 = min(N, row0 + rpm);
        float* a_sm = stages;                         // N floats (N <= 16384: two stages)
        float* dr = stages + 16384;                   // up to N floats
        for (int l = L; l >= 1; --l) {
            const int depth = L - l + P.depth_shift;
            if (depth % P.shard_count != P.shard_rank) continue;        // another shard's layer
            if ((((depth / P.shard_count) % P.keff) % G) != g) continue;   // not a layer of my group
            if (row0 < row1) worker_store_rows<UPDATE>(P, l, row0, row1, dr, a_sm, sh);
        }
        cluster_sync_all();   // the cluster's CTAs leave together
        return;
    }

    // ===================== chain clusters ====================================================
    const int q = cluster_id;
    const int Wc = P.Wc, nCB = P.nCB, R = P.R, nRB = P.nRB, Hr = P.Hr, Ws = P.Ws;
    const int WC4 = Wc >> 2;
    const int RG = PK_CHAIN_THREADS / WC4;    // row groups of the 128 threads of either half
    const int ht = tid & (PK_CHAIN_THREADS - 1);   // thread index inside its half (chain / store)
    const int tcol = ht % WC4, trow = ht / WC4;
    const int row_base = c * Hr;
    const int row_end = min(N, row_base + Hr);
    const int col_base = q * Ws;
    const int Hr_pad = nRB * R;

    if (warp == PK_PRODUCER_WARP) {
        // ------------------------- producer: weight sub-tiles by TMA, ahead of the chain ---------
        // Issuing a tensor copy costs its thread several hundred cycles; on a thread of the chain
        // warps that was a sixth of every layer step.  Here it costs nothing: lane 0 waits until
        // the chain warps (and, under the fused weight update, the store warps) are done with a
        // stage and refills it.
        if (lane == 0) {
            const int nSub = nCB * nRB;
            const int total = (L - 1) * nSub;
            const unsigned stage_bytes = (unsigned)(R * Wc * sizeof(float));
            int is_s = L, is_cb = 0, is_rb = 0, is_it = 0;   // the next sub-tile: layer, column block, row block
            for (; is_it < total; ++is_it) {
                const int st = is_it % PK_STAGES;
                if (is_it >= PK_STAGES) {
                    const unsigned parity = (unsigned)(((is_it / PK_STAGES) - 1) & 1);
                    wait_bar<false>(smem_u32(&sh->empty[st]), parity, P, sh);
                    if (UPDATE && P.fused) wait_bar<false>(smem_u32(&sh->st_done[st]), parity, P, sh);
                    if (sh->abort_flag) break;
                }
                const unsigned bar = smem_u32(&sh->full[st]);
                mbar_expect_tx(bar, stage_bytes);
                tma_load_3d(smem_u32(stages + (size_t)st * PK_STAGE_FLOATS), &w_map, bar,
                            col_base + is_cb * Wc, row_base + is_rb * R, is_s - 1);
                if (++is_rb == nRB) { is_rb = 0; if (++is_cb == nCB) { is_cb = 0; --is_s; } }
            }
            // A CTA that gave up waiting may still have weight tiles on their way into its shared
            // memory; it must not exit under them.  Wait for the last loads, with a limit.
            if (sh->abort_flag) {
                const unsigned long long t0 = globaltimer_ns();
                for (int j = is_it > PK_STAGES ? is_it - PK_STAGES : 0; j < is_it; ++j) {
                    const unsigned bar = smem_u32(&sh->full[j % PK_STAGES]);
                    const unsigned parity = (unsigned)((j / PK_STAGES) & 1);
                    while (!mbar_try_wait(bar, parity) && globaltimer_ns() - t0 < 50000000ull) { }
                }
            }
        }
    } else if (warp >= PK_CHAIN_WARPS) {
        // ------------------------- store warps: gw^s = delta^s (x) a^{s-1} ---------------------
        if (P.fused) {
            float4 a4[PK_MAX_NCB], a4_next[PK_MAX_NCB];
            auto load_a4 = [&](int l, float4* dst) {
                const float* av = P.a + (size_t)l * N;
#pragma unroll
                for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
                    dst[cb] = make_float4(0.f, 0.f, 0.f, 0.f);
                    const int col = col_base + cb * Wc + tcol * 4;
                    if (cb < nCB && col < N) dst[cb] = *reinterpret_cast<const float4*>(av + col);
                }
            };
            load_a4(L - 1, a4);
            int it_store = 0;   // running sub-tile index, the chain warps' `it`
            for (int s = L; s >= 1; --s) {
                const int p = s & 1;
                const unsigned use = (unsigned)((L - s) >> 1);      // how often buffer p was used before
                if (s >= 2) load_a4(s - 2, a4_next);
                wait_bar<false>(smem_u32(&sh->d_ready[p]), use & 1u, P, sh);
                const float* dr = d_rows + p * PK_DROWS;
                float* gw_s = P.gw + (size_t)(s - 1) * N * N;
                // layer-sharded form: the tile of another shard's layer is not stored; every wait and
                // arrival below still takes place, so the chain and the producer see no difference
                const bool mine = (L - s + P.depth_shift) % P.shard_count == P.shard_rank;
                if (UPDATE && s >= 2) {
                    // Fused weight update, layers the chain reads: the sub-tiles of w^s pass through
                    // this CTA's shared memory for the chain anyway, so the store warps take w from
                    // there (the same stage, the same element mapping as the chain warps) -- no second
                    // read of w from memory -- and tell the producer when they are done with a stage.
                    const int rows = row_end - row_base;
#pragma unroll
                    for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
                        if (cb >= nCB) break;
                        const int col = col_base + cb * Wc + tcol * 4;
                        const float4 av = a4[cb];
                        float* out = gw_s + (size_t)row_base * N + col;
                        for (int rb = 0; rb < nRB; ++rb, ++it_store) {
                            const int st = it_store % PK_STAGES;
                            wait_bar<false>(smem_u32(&sh->full[st]), (unsigned)((it_store / PK_STAGES) & 1), P, sh);
                            const float4* tile = reinterpret_cast<const float4*>(stages + (size_t)st * PK_STAGE_FLOATS);
                            if (mine && col < N) {
#pragma unroll 8
                                for (int i = 0; i < 16; ++i) {
                                    const int rr = rb * R + trow + i * RG;
                                    if (rr < rows) {
                                        const float d = dr[rr];
                                        st_stream4(out + (size_t)rr * N,
                                                   lf_sgd_apply4(P.eta, tile[ht + i * PK_CHAIN_THREADS],
                                                                 make_float4(d * av.x, d * av.y, d * av.z, d * av.w)));
                                    }
                                }
                            }
                            mbar_arrive(smem_u32(&sh->st_done[st]));
                        }
                    }
                    mbar_arrive(smem_u32(&sh->d_free[p]));
#pragma unroll
                    for (int cb = 0; cb < PK_MAX_NCB; ++cb) a4[cb] = a4_next[cb];
                    continue;
                }
#pragma unroll
                for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
                    if (cb >= nCB || !mine) break;
                    const int col = col_base + cb * Wc + tcol * 4;
                    if (col >= N) continue;
                    const float4 av = a4[cb];
                    float* out = gw_s + (size_t)row_base * N + col;
                    const int rows = row_end - row_base;
                    if (UPDATE) {
                        // fused update of layer 1, which the chain never reads: w^1 comes from memory
                        store_tile_updated(P.w_sub + (size_t)(s - 1) * N * N + (size_t)row_base * N + col, out, dr, av,
                                           rows, trow, RG, N, P.eta);
                    } else {
#pragma unroll 4
                        for (int rr = trow; rr < rows; rr += RG) {
                            const float d = dr[rr];
                            st_stream4(out + (size_t)rr * N, make_float4(d * av.x, d * av.y, d * av.z, d * av.w));
                        }
                    }
                }
                mbar_arrive(smem_u32(&sh->d_free[p]));
#pragma unroll
                for (int cb = 0; cb < PK_MAX_NCB; ++cb) a4[cb] = a4_next[cb];
            }
        }
    } else {
        // ------------------------- chain warps --------------------------------------------------
        const int wpr = WC4 > 32 ? WC4 / 32 : 1;   // warps that share one tile row

        const int my_col = col_base + c * P.slice + tid;   // the column this thread finishes (tid < slice)
        const bool finisher = tid < P.slice && my_col < N;
        float a_mine = finisher ? P.a[(size_t)(L - 1) * N + my_col] : 0.f;

        // ---- Eq. bp1: delta^L for my rows (every cluster computes it for itself)
        {
            const float* aL = P.a + (size_t)L * N;
            float* dr = d_rows + (L & 1) * PK_DROWS;
            for (int r = tid; r < Hr_pad; r += PK_CHAIN_THREADS) {
                const int row = row_base + r;
                float d = 0.f;
                if (r < Hr && row < N) {
                    if (P.top_given) {
                        d = P.delta[(size_t)(L - 1) * N + row];   // written (with gb) by an earlier launch
                    } else {
                        const float av = aL[row];
                        d = av - P.y[row];
                        if (P.cost == LF_COST_QUADRATIC) d *= lf_act_prime(av, P.act);   // cross-entropy: sigma' cancels
                        if (q == 0) {
                            P.delta[(size_t)(L - 1) * N + row] = d;
                            P.gb[(size_t)(L - 1) * N + row] = d;                  // Eq. bp3
                        }
                    }
                    if (q == 0 && P.Qw > 0) st_slot(P.xch + (size_t)(L - 1) * N + row, d, P.epoch);
                }
                dr[r] = d;
            }
            mbar_arrive(smem_u32(&sh->d_ready[L & 1]));
        }
        chain_sync();

        // With one column block and at most 32 columns to finish per CTA the four chain warps
        // send their partial sums straight to the finishing CTA (recv then holds C*4 rows of 32).
        const bool direct = nCB == 1 && WC4 <= 32 && P.slice <= 32;   // (every warp must span the whole strip)
        int it = 0;
        for (int s = L; s >= 2; --s) {
            PK_STAMP(0);
            const int p = s & 1;
            const float* dr = d_rows + p * PK_DROWS;
            float* recv_p = recv + p * PK_MAX_CLUSTER * PK_MAX_SLICE;
            const float a_mine_next = (finisher && s >= 3) ? P.a[(size_t)(s - 2) * N + my_col] : 0.f;
            // this step's partial sums for my slice will be credited: slice floats from every
            // CTA of the cluster (from each of its four chain warps on the direct path)
            if (tid == 0)
                mbar_expect_tx(smem_u32(&sh->part_ready[p]),
                               (unsigned)(C * P.slice * sizeof(float)) * (direct ? PK_CHAIN_WARPS : 1));

#pragma unroll
            for (int cb = 0; cb < PK_MAX_NCB; ++cb) {
                if (cb >= nCB) break;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                float4* red_p = red + (cb & 1) * PK_CHAIN_THREADS;
                for (int rb = 0; rb < nRB; ++rb, ++it) {
                    const int st = it % PK_STAGES;
                    wait_bar<false>(smem_u32(&sh->full[st]), (unsigned)((it / PK_STAGES) & 1), P, sh);
                    if (rb == 0 && cb == 0) PK_STAMP(1);
                    const float4* tile = reinterpret_cast<const float4*>(stages + (size_t)st * PK_STAGE_FLOATS);
                    const float* drb = dr + rb * R + trow;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        // row trow + i*RG of the sub-tile; RG * WC4 == 128, so the float4 index is
                        const float4 wv = tile[tid + i * PK_CHAIN_THREADS];
                        const float d = drb[i * RG];
                        acc.x = fmaf(wv.x, d, acc.x);
                        acc.y = fmaf(wv.y, d, acc.y);
                        acc.z = fmaf(wv.z, d, acc.z);
                        acc.w = fmaf(wv.w, d, acc.w);
                    }
                    if (rb == nRB - 1) {
                        // partial column sums of this column block: first the row groups that
                        // share a warp (shuffles, fixed order), then one entry per warp
                        for (int off = WC4; off < 32; off <<= 1) {
                            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, off);
                            acc.y += __shfl_xor_sync(0xffffffffu, acc.y, off);
                            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, off);
                            acc.w += __shfl_xor_sync(0xffffffffu, acc.w, off);
                        }
                        if (direct) {
                            // narrow strip: every warp hands its own partial sums to the finishing CTA
                            if (lane < WC4) {
                                const int cs = lane * 4;
                                const int owner = cs / P.slice, off = cs - owner * P.slice;
                                st_async_f32x4(map_to_cta(smem_u32(recv_p + (c * PK_CHAIN_WARPS + warp) * 32 + off),
                                                          (unsigned)owner),
                                               acc, map_to_cta(smem_u32(&sh->part_ready[p]), (unsigned)owner));
                            }
                        } else if (lane < WC4) {
                            red_p[warp * 32 + lane] = acc;
                        }
                    }
                    // this warp is done with the stage: tell the producer (no CTA-wide barrier per
                    // sub-tile; only the entries in red_p need one, at the end of a column block)
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh->empty[st]));
                    if (rb == nRB - 1 && !direct) chain_sync();   // red_p is complete
                }
                if (cb == 0) PK_STAMP(2);
                if (!direct && tid < WC4) {
                    // add the warps' entries in order; warps (tid>>5), +wpr, ... hold my columns
                    const int l5 = tid & 31;
                    int wq = tid >> 5;
                    float4 sum = red_p[wq * 32 + l5];
                    for (wq += wpr; wq < PK_CHAIN_WARPS; wq += wpr) {
                        const float4 t = red_p[wq * 32 + l5];
                        sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
                    }
                    // hand the four columns to the CTA that finishes them and tell it
                    const int cs = cb * Wc + tid * 4;            // column inside the strip
                    const int owner = cs / P.slice, off = cs - owner * P.slice;
                    st_async_f32x4(map_to_cta(smem_u32(recv_p + c * PK_MAX_SLICE + off), (unsigned)owner), sum,
                                   map_to_cta(smem_u32(&sh->part_ready[p]), (unsigned)owner));
                }
            }
            PK_STAMP(3);
            // the partial sums for my slice of the strip, from every CTA of the cluster
            wait_bar<true>(smem_u32(&sh->part_ready[p]), (unsigned)(((L - s) >> 1) & 1), P, sh);
            PK_STAMP(4);
            if (tid < P.slice) {
                // add the partial sums in a fixed order (loads issued together, adds in sequence)
                const int n_src = direct ? C * PK_CHAIN_WARPS : C;
                const int src_ld = direct ? 32 : PK_MAX_SLICE;
                float part[PK_MAX_CLUSTER * PK_CHAIN_WARPS];
#pragma unroll
                for (int cc = 0; cc < PK_MAX_CLUSTER * PK_CHAIN_WARPS; ++cc)
                    part[cc] = cc < n_src ? recv_p[cc * src_ld + tid] : 0.f;
                float v = part[0];
#pragma unroll
                for (int cc = 1; cc < PK_MAX_CLUSTER * PK_CHAIN_WARPS; ++cc)
                    if (cc < n_src) v += part[cc];
                if (my_col < N) {
                    const float d = v * lf_act_prime(a_mine, P.act);   // Eq. bp2
                    if (!(P.withhold && blockIdx.x == 0)) st_slot(P.xch + (size_t)(s - 2) * N + my_col, d, P.epoch);
                    P.delta[(size_t)(s - 2) * N + my_col] = d;
                    P.gb[(size_t)(s - 2) * N + my_col] = d;           // Eq. bp3
                }
            }
            a_mine = a_mine_next;
            PK_STAMP(5);
            // delta^{s-1} of my rows, from whichever clusters finished those columns, into the
            // other delta buffer once the store warps have let go of it
            {
                const int pn = (s - 1) & 1;
                const unsigned used = (unsigned)((L - (s - 1)) >> 1);   // earlier uses of buffer pn
                if (P.fused && used > 0) wait_bar<false>(smem_u32(&sh->d_free[pn]), (used - 1) & 1u, P, sh);
                float* dn = d_rows + pn * PK_DROWS;
                const unsigned long long* slots = P.xch + (size_t)(s - 2) * N;
                for (int r0 = 0; r0 < Hr_pad; r0 += 4 * PK_CHAIN_THREADS) {
                    unsigned long long v[4];
                    bool pend[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {      // up to four polls in flight per thread
                        const int r = r0 + u * PK_CHAIN_THREADS + tid;
                        pend[u] = r < Hr && row_base + r < N;
                        v[u] = pend[u] ? ld_slot(slots + row_base + r) : 0ull;
                    }
                    // poll whatever is still missing, all of it together, until it is there
                    unsigned long long t0 = 0;
                    unsigned rounds = 0;
                    for (;;) {
                        bool any = false;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (pend[u]) {
                                if ((unsigned)(v[u] >> 32) == P.epoch) pend[u] = false;
                                else { v[u] = ld_slot(slots + row_base + r0 + u * PK_CHAIN_THREADS + tid); any = true; }
                            }
                        }
                        if (!any) break;
                        bool give_up = sh->abort_flag != 0u;
                        if (!give_up && (++rounds & 15u) == 0u) {
                            const unsigned long long now = globaltimer_ns();
                            if (t0 == 0) t0 = now;
                            if (now - t0 > P.budget_ns || *((volatile unsigned*)P.status) != 0u) {
                                raise_timeout(P, sh, LF_DEV_TIMEOUT_FLAG);
                                give_up = true;
                            }
                        }
                        if (give_up) {
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (pend[u]) v[u] = 0ull;
                            break;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int r = r0 + u * PK_CHAIN_THREADS + tid;
                        if (r < Hr_pad) dn[r] = __uint_as_float((unsigned)v[u]);
                    }
                }
                mbar_arrive(smem_u32(&sh->d_ready[pn]));
            }
            chain_sync();
            PK_STAMP(6);
        }
    }
    __syncthreads();
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

constexpr size_t PK_SMEM_BYTES = (size_t)PK_STAGES * PK_STAGE_FLOATS * 4 + (size_t)2 * PK_DROWS * 4 +
                                 2 * PK_CHAIN_THREADS * 16 + 2 * PK_MAX_CLUSTER * PK_MAX_SLICE * 4 + 256;
static_assert(sizeof(PkShared) <= 256, "the barrier block must fit into the space reserved for it");

struct PkPlan {
    bool ok;
    int C, Qmax, Qc, Qw, Wc, nCB, Ws, Hr, R, nRB, slice;
};

void cluster_launch_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* at, int C, int clusters)
{
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3(C * clusters);
    cfg->blockDim = dim3(PK_LAUNCH_THREADS);
    cfg->dynamicSmemBytes = PK_SMEM_BYTES;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg->attrs = at; cfg->numAttrs = 1;
}

// How many clusters of C CTAs (one CTA per SM at this shared-memory size) fit on the device.
int max_active_clusters(const lf_ctx* c, int C)
{
    static int cached_dev = -1, cached[PK_MAX_CLUSTER + 1];
    if (cached_dev != c->device) {
        for (int i = 0; i <= PK_MAX_CLUSTER; ++i) cached[i] = -1;
        cached_dev = c->device;
    }
    if (cached[C] >= 0) return cached[C];
    int n = 0;
    if (cudaFuncSetAttribute(k_backward_persistent<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)PK_SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(k_backward_persistent<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)PK_SMEM_BYTES) == cudaSuccess) {
        cudaLaunchConfig_t cfg; cudaLaunchAttribute at[1];
        cluster_launch_config(&cfg, at, C, 16);
        int n_upd = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_backward_persistent<false>, &cfg) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n_upd, k_backward_persistent<true>, &cfg) != cudaSuccess)
            n = 0;
        else if (n_upd < n)
            n = n_upd;
    }
    cudaGetLastError();
    cached[C] = n;
    return n;
}

PkPlan plan_for_cluster(const lf_ctx* c, int variant, int C)
{
    PkPlan p = {};
    p.C = C;
    p.Qmax = max_active_clusters(c, C);
    int Qc_budget = p.Qmax;
    if (variant == LF_VARIANT_PERSISTENT) {
        if (p.Qmax < 2) return p;
        // Half of the clusters for the chain, half for the workers; a shard stores only every S-th
        // layer, so its workers get by with 1 / (S + 1) of the clusters.
        Qc_budget = p.Qmax / 2;
        if (c->shard_count > 1) {
            int workers = p.Qmax / (c->shard_count + 1);
            if (workers < 1) workers = 1;
            Qc_budget = p.Qmax - workers;
        }
    }
    if (Qc_budget < 1) return p;
    const int N = c->pk_N;
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
    p.Hr = (N + C - 1) / C;
    p.nRB = (p.Hr + p.R - 1) / p.R;
    p.slice = p.Ws / C;
    if (p.slice > PK_MAX_SLICE || p.slice < 4 || p.nRB * p.R > PK_DROWS) return p;
    if (variant == LF_VARIANT_PERSISTENT && N > 16384) return p;
    p.ok = true;
    return p;
}

// Pick the cluster size that puts the most CTAs (SMs) on the delta chain -- the chain sets the pace
// (measured for the leapfrog groups at N = 256..2048: the cluster size with the most chain CTAs was
// the fastest or within 2 % of it, however many workers it left); ties go to the larger cluster,
// whose CTAs hold fewer rows each.
PkPlan make_plan(const lf_ctx* c, int variant)
{
    PkPlan best = {};
    if (c->B != 1 || c->pk_N <= 0 || c->pk_L < 1) return best;
    if ((size_t)c->smem_optin < PK_SMEM_BYTES) return best;
    if (!get_encode_fn()) return best;
    int best_ctas = 0;
    for (int C = PK_MAX_CLUSTER; C >= 2; C >>= 1) {
        PkPlan p = plan_for_cluster(c, variant, C);
        if (!p.ok) continue;
        const int ctas = p.Qc * C;
        if (ctas > best_ctas) { best = p; best_ctas = ctas; }
    }
    return best;
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
    if (variant == LF_VARIANT_FUSED && lf_columns_supported(c)) return true;
    return make_plan(c, variant).ok;
}

// Which of the two fused kernels serves a context: whole columns per CTA (one hop per layer), or
// cluster tiles.  The same rule holds for the plain pass and for the fused weight update, so that
// the two give the same gradients bit for bit.
int lf_fused_tiling(const lf_ctx* c)
{
    const bool columns_ok = lf_columns_supported(c);
    const bool clusters_ok = make_plan(c, LF_VARIANT_FUSED).ok;
    if (c->opt_fused_tiling == LF_FUSED_TILING_COLUMNS && columns_ok) return LF_FUSED_TILING_COLUMNS;
    if (c->opt_fused_tiling == LF_FUSED_TILING_CLUSTERS && clusters_ok) return LF_FUSED_TILING_CLUSTERS;
    if (columns_ok && (!clusters_ok || c->pk_N <= LF_COLUMNS_FUSED_MAX_N)) return LF_FUSED_TILING_COLUMNS;
    return LF_FUSED_TILING_CLUSTERS;
}

// LF_VARIANT_AUTO for one sample: fused pass or leapfrog CTA groups, from measurement (B200, L = 32,
// buffers rotated so that nothing is found in L2, N = 256..4096, k = 1..8).  Up to N = 2048 the pass
// is bound by the delta hand-off.  Up to N = 640 the fused pass with whole columns per CTA -- one
// hop per layer, few CTAs -- is 3-12 % ahead of everything else.  From there to N = 2048 the groups
// variant -- whose chain has half of the clusters, hence wider strips and fewer CTAs to wait for,
// and stores nothing itself -- is 1-12 % ahead with up to four workers; with more workers (fewer
// CTAs per layer) only at the widths listed.  From N = 2560 the pass is bandwidth-bound and the fused
// pass, which leaves no SM without a share of the weights, is 4-8 % ahead.
int lf_auto_variant(const lf_ctx* c)
{
    if (c->B != 1 || c->pk_N <= 0) return LF_VARIANT_STREAMS;
    const int N = c->pk_N;
    if (N <= LF_COLUMNS_AUTO_MAX_N && lf_columns_supported(c)) return LF_VARIANT_FUSED;
    const bool groups_faster = c->keff <= 4 ? N <= 2048 : (N <= 576 || (N >= 832 && N <= 1280));
    if (groups_faster && make_plan(c, LF_VARIANT_PERSISTENT).ok) return LF_VARIANT_PERSISTENT;
    return lf_persistent_supported(c, LF_VARIANT_FUSED) ? LF_VARIANT_FUSED : LF_VARIANT_STREAMS;
}

// The launch covers the pk_L layers of width pk_N that w, a, delta, gw, gb (and w_sub) point at --
// the whole network, or the run of equal-width layers in its middle (top_given, depth_shift = 1).
int lf_backward_persistent(lf_ctx* c, int variant, const float* w, const float* a, const float* y, float* delta,
                           float* gw, float* gb, const float* w_sub, int top_given, int depth_shift)
{
    const int L_run = c->pk_L, N_run = c->pk_N;
    c->stats.fused_tiling = 0;
    if (variant == LF_VARIANT_FUSED && lf_fused_tiling(c) == LF_FUSED_TILING_COLUMNS) {
        c->stats.fused_tiling = LF_FUSED_TILING_COLUMNS;
        return lf_backward_columns(c, w, a, y, delta, gw, gb, w_sub, top_given, depth_shift);
    }
    PkPlan pl = make_plan(c, variant);
    if (!pl.ok) return LF_ERESOURCE;
    if (variant == LF_VARIANT_FUSED) c->stats.fused_tiling = LF_FUSED_TILING_CLUSTERS;
    // tensor map over w as [L][N][N], box = Wc columns x R rows x 1 layer
    if (!c->w_map_valid || c->w_map_ptr != w || c->w_map_wc != pl.Wc) {
        CUtensorMap* m = reinterpret_cast<CUtensorMap*>(c->w_map_storage);
        cuuint64_t dims[3] = {(cuuint64_t)N_run, (cuuint64_t)N_run, (cuuint64_t)L_run};
        cuuint64_t strides[2] = {(cuuint64_t)N_run * 4, (cuuint64_t)N_run * N_run * 4};
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
    P.L = L_run; P.N = N_run; P.C = pl.C; P.Qc = pl.Qc; P.Qw = pl.Qw;
    P.top_given = top_given; P.depth_shift = depth_shift;
    P.fused = variant == LF_VARIANT_FUSED ? 1 : 0;
    P.Wc = pl.Wc; P.nCB = pl.nCB; P.Ws = pl.Ws; P.Hr = pl.Hr; P.R = pl.R; P.nRB = pl.nRB;
    P.slice = pl.slice; P.keff = c->keff; P.epoch = c->epoch; P.withhold = c->withhold == 1 ? 1 : 0;
    P.cost = c->opt_cost; P.act = c->opt_act;
    P.shard_rank = c->shard_rank; P.shard_count = c->shard_count > 1 ? c->shard_count : 1;
    P.budget_ns = (unsigned long long)c->wait_budget_us * 1000ull;
    P.a = a; P.y = y; P.delta = delta; P.gw = gw; P.gb = gb;
    P.w_sub = c->sgd_on ? w_sub : nullptr; P.eta = c->sgd_eta;
    P.xch = reinterpret_cast<unsigned long long*>(c->sync_words);
    P.status = c->status_dev;
#ifdef LF_PK_TRACE
    if (!c->trace_dev) cudaMalloc(&c->trace_dev, (size_t)2 * c->L * 16 * sizeof(unsigned long long));
    cudaMemsetAsync(c->trace_dev, 0, (size_t)2 * c->L * 16 * sizeof(unsigned long long), c->stream);
    P.trace = c->trace_dev;
#endif

    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_persistent<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)PK_SMEM_BYTES));
    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_persistent<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)PK_SMEM_BYTES));
    cudaLaunchConfig_t cfg; cudaLaunchAttribute at[1];
    cluster_launch_config(&cfg, at, pl.C, pl.Qc + pl.Qw);
    cfg.stream = c->stream;
    const CUtensorMap* mp = reinterpret_cast<const CUtensorMap*>(c->w_map_storage);
    if (P.w_sub)
        LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_persistent<true>, *mp, P));
    else
        LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_persistent<false>, *mp, P));
    c->stats.launches_backward = 1;
    c->stats.chain_ctas = pl.Qc * pl.C;
    c->stats.worker_ctas = pl.Qw * pl.C;
    return LF_OK;
}

void lf_persistent_release(lf_ctx* c)
{
#if defined(LF_PK_TRACE) || defined(LF_CK_TRACE)
    if (c->trace_dev) cudaFree(c->trace_dev);
#else
    (void)c;
#endif
}

#if defined(LF_PK_TRACE) || defined(LF_CK_TRACE)
// Debug builds: copy the SM-clock stamps of the last persistent launch to `out` (2 * L * 16 words).
extern "C" int lf_debug_read_trace(lf_ctx* c, unsigned long long* out)
{
    if (!c || !out || !c->trace_dev) return LF_ENULL;
    cudaStreamSynchronize(c->stream);
    return cudaMemcpy(out, c->trace_dev, (size_t)2 * c->L * 16 * sizeof(unsigned long long),
                      cudaMemcpyDeviceToHost) == cudaSuccess ? LF_OK : LF_ECUDA;
}
#endif
