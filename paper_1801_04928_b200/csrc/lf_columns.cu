// Fused single-launch backward pass for one sample (B = 1) with WHOLE COLUMNS per CTA.
//
// The delta recurrence (Eq. bp2) is sequential in depth, and at widths of about a thousand a layer
// holds so little data that a pass is bound by how fast delta^{l+1} gets from the CTAs that finish
// it to the CTAs that need it, not by memory bandwidth.  This kernel keeps that hand-off to ONE hop
// through L2 per layer:
//
//   * CTA q owns the columns [q*Wc, (q+1)*Wc) of every weight matrix -- all N rows of them -- so the
//     column sums  t_k = sum_j w^s_jk delta^s_j  of its columns are complete inside the CTA: no
//     partial sums cross CTAs.  It applies sigma' and publishes its Wc values of delta^{s-1} as
//     8-byte {value, epoch} slots; every CTA polls all N slots of a layer.
//   * The eight CHAIN WARPS split the rows of each weight sub-tile between them.  A warp polls
//     exactly the delta values of its own rows and multiplies as soon as IT has them: no CTA-wide
//     barrier sits between the arrival of delta and the multiply.  One barrier per layer joins the
//     warps' partial sums (shuffles inside a warp, shared memory across warps, fixed order).
//   * Weight tiles do not depend on delta: a producer warp streams them by TMA through a ring of
//     shared-memory stages, several layers ahead of the chain at small widths.
//   * The Wc values of delta^l a CTA finishes are rows [q*Wc, (q+1)*Wc) of gw^l = delta^l (x)
//     a^{l-1} (Eq. bp4), known there first.  Four STORE WARPS stream those rows out -- whole rows,
//     128-bit streaming stores -- while the chain goes on; they never touch the weight tiles.  The
//     chain may run two layers ahead of the stores (two delta buffers), not more.
//
// Every wait is bounded by a time budget.  On expiry the CTA raises the status word, stops waiting
// for the rest of the launch and runs to the end with whatever it has, so the kernel always ends.
#include <cuda.h>
#include <string.h>

#include "lf_internal.h"
#include "lf_ptx.cuh"

namespace {

using namespace lfptx;

constexpr int CK_CHAIN_WARPS = 8;
constexpr int CK_CHAIN_THREADS = 32 * CK_CHAIN_WARPS;
constexpr int CK_STORE_WARPS = 4;
constexpr int CK_STORE_THREADS = 32 * CK_STORE_WARPS;
constexpr int CK_PRODUCER_WARP = CK_CHAIN_WARPS + CK_STORE_WARPS;
constexpr int CK_THREADS = 32 * (CK_PRODUCER_WARP + 1);
#ifndef CK_MIN_WC
#define CK_MIN_WC 8                       // fewest columns per CTA
#endif
constexpr int CK_MAX_WC = 128;            // columns per CTA: a multiple of 4, at most 32 float4 per row
constexpr int CK_MAX_STAGES = 24;
constexpr int CK_STAGE_FLOATS = 8192;     // a sub-tile (one TMA box) holds at most 32 KiB
constexpr int CK_POLL_BATCH = 4;          // slots a thread polls at a time
constexpr int CK_MAX_N = 16384;
constexpr size_t CK_SMEM_LIMIT = 227 * 1024;

struct CkParams {
    int L, N;
    int Q;             // CTAs = column strips
    int Wc;            // columns per CTA
    int RL, RH;        // TMA box: RL rows (a divisor of N) times RH row blocks
    int R;             // rows per sub-tile = RL * RH
    int nSub;          // sub-tiles per layer
    int Rw;            // rows of a sub-tile per chain warp
    int stages;        // ring depth
    int stage_floats;  // ring stride (the box, rounded up to 128 bytes)
    int shard_rank, shard_count, top_given, depth_shift;   // as in the cluster kernel
    int withhold, cost, act;
    unsigned epoch;
    unsigned long long budget_ns;
    const float* a;
    const float* y;
    const float* w_sub;        // fused weight update: store w_sub - eta * gw in place of gw (null: plain gw)
    float eta;
    float* delta;
    float* gw;
    float* gb;
    unsigned long long* xch;   // [L][N] slots
    unsigned* status;
#ifdef LF_CK_TRACE
    unsigned long long* trace;  // [2 CTAs][L][8] SM-clock stamps (debug builds only)
#endif
};

struct CkShared {
    unsigned long long full[CK_MAX_STAGES];    // TMA arrival
    unsigned long long empty[CK_MAX_STAGES];   // the chain warps have read the stage
    unsigned long long d_ready[2];             // finished delta values of a layer are in d_own[p]
    unsigned long long d_free[2];              // the store warps are done with d_own[p]
    volatile unsigned abort_flag;
};

#ifdef LF_CK_TRACE
#define CK_STAMP(slot)                                                                            \
    do {                                                                                          \
        if (tid == 0 && (blockIdx.x == 0 || blockIdx.x == (unsigned)(P.Q / 2 + 1)))               \
            P.trace[((blockIdx.x == 0 ? 0 : 1) * (size_t)P.L + (size_t)(P.L - s)) * 8 + (slot)] = \
                (unsigned long long)clock64();                                                    \
    } while (0)
#else
#define CK_STAMP(slot) do { } while (0)
#endif

__device__ __forceinline__ void ck_raise(const CkParams& P, CkShared* sh, unsigned bit)
{
    atomicOr(P.status, bit);
    sh->abort_flag = 1u;
}

__device__ __forceinline__ void ck_wait(unsigned bar, unsigned parity, const CkParams& P, CkShared* sh)
{
    if (mbar_try_wait(bar, parity)) return;
    if (sh->abort_flag) return;
    const unsigned long long t0 = globaltimer_ns();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 15u) == 0u) {
            if (sh->abort_flag) return;
            if (globaltimer_ns() - t0 > P.budget_ns) {
                ck_raise(P, sh, LF_DEV_TIMEOUT_BARRIER);
                return;
            }
        }
    }
}

// Eq. bp1 at one neuron of the top layer (or delta^L as an earlier launch left it); aL, deltaL: the
// top layer's activations and delta.
__device__ __forceinline__ float ck_top_delta_at(const CkParams& P, const float* aL, const float* deltaL, int row)
{
    if (P.top_given) return deltaL[row];
    const float av = aL[row];
    float d = av - P.y[row];
    if (P.cost == LF_COST_QUADRATIC) d *= lf_act_prime(av, P.act);   // cross-entropy: sigma' cancels
    return d;
}
__device__ __forceinline__ float ck_top_delta(const CkParams& P, int row)
{
    return ck_top_delta_at(P, P.a + (size_t)P.L * P.N, P.delta + (size_t)(P.L - 1) * P.N, row);
}

// Polling delta^s at the rows this warp multiplies (d_sm index = row; rows past N hold 0).  A lane
// polls up to CK_POLL_BATCH slots at a time: the loads of a batch are issued together and collected
// together, so a batch costs one round trip to L2 when the values are there.
struct CkPoll {
    int row[CK_POLL_BATCH];
    bool valid[CK_POLL_BATCH], pend[CK_POLL_BATCH];
    unsigned long long v[CK_POLL_BATCH];
    int sub, piece;      // the next item (counted up, never divided: this is the chain)
};

// rows of the next batch (R rows per sub-tile, Rw of them this warp's, nSub sub-tiles, n_rows rows in all)
__device__ __forceinline__ void ck_poll_setup(CkPoll& q, int R, int Rw, int nSub, int n_rows, int warp, int lane)
{
    const int cpw = (Rw + 31) >> 5;               // 32-row pieces of a warp's share of a sub-tile
#pragma unroll
    for (int u = 0; u < CK_POLL_BATCH; ++u) {
        const int off = q.piece * 32 + lane;
        const int rl = warp * Rw + off;
        q.row[u] = q.sub * R + rl;
        q.valid[u] = q.sub < nSub && off < Rw && rl < R;
        if (++q.piece == cpw) { q.piece = 0; ++q.sub; }
        q.pend[u] = q.valid[u] && q.row[u] < n_rows;
        q.v[u] = 0ull;
    }
}
__device__ __forceinline__ void ck_poll_issue(CkPoll& q, const unsigned long long* slots)
{
#pragma unroll
    for (int u = 0; u < CK_POLL_BATCH; ++u)
        if (q.pend[u]) q.v[u] = ld_slot(slots + q.row[u]);
}
// wait until every slot of the batch carries this call's epoch (re-polling what does not), then
// put the values into d_sm
__device__ __forceinline__ void ck_poll_collect(CkPoll& q, const CkParams& P, CkShared* sh,
                                                const unsigned long long* slots, float* d_sm)
{
    unsigned long long t0 = 0;
    unsigned rounds = 0;
    for (;;) {
        bool any = false;
#pragma unroll
        for (int u = 0; u < CK_POLL_BATCH; ++u) {
            if (q.pend[u]) {
                if ((unsigned)(q.v[u] >> 32) == P.epoch) q.pend[u] = false;
                else { q.v[u] = ld_slot(slots + q.row[u]); any = true; }
            }
        }
        if (!any) break;
        bool give_up = sh->abort_flag != 0u;
        if (!give_up && (++rounds & 15u) == 0u) {
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > P.budget_ns || *((volatile unsigned*)P.status) != 0u) {
                ck_raise(P, sh, LF_DEV_TIMEOUT_FLAG);
                give_up = true;
            }
        }
        if (give_up) {
#pragma unroll
            for (int u = 0; u < CK_POLL_BATCH; ++u)
                if (q.pend[u]) { q.pend[u] = false; q.v[u] = 0ull; }
            break;
        }
    }
#pragma unroll
    for (int u = 0; u < CK_POLL_BATCH; ++u)
        if (q.valid[u]) d_sm[q.row[u]] = __uint_as_float((unsigned)q.v[u]);
}

// UPDATE = true: the instance behind lf_backward_sgd (P.w_sub set).  Its store warps read the rows
// of w they update from memory: those are not the columns the chain has in shared memory.
template <bool UPDATE>
__global__ void __launch_bounds__(CK_THREADS, 1)
k_backward_columns(const __grid_constant__ CUtensorMap w_map, const CkParams P)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    float* ring = reinterpret_cast<float*>(smem_raw);                                // stages x stage_floats
    float* d_sm = ring + (size_t)P.stages * P.stage_floats;                          // [nSub * R]
    float4* red = reinterpret_cast<float4*>(d_sm + (((size_t)P.nSub * P.R + 3) & ~(size_t)3));   // [2][8 warps][32]
    float* d_own = reinterpret_cast<float*>(red + 2 * CK_CHAIN_WARPS * 32);          // [2][CK_MAX_WC]
    CkShared* sh = reinterpret_cast<CkShared*>(d_own + 2 * CK_MAX_WC);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = P.N, L = P.L, Wc = P.Wc;
    const int col_base = blockIdx.x * Wc;
    const int my_cols = min(Wc, N - col_base);   // >= 4

    if (tid == 0) {
        for (int i = 0; i < P.stages; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->empty[i]), CK_CHAIN_WARPS);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh->d_ready[i]), (unsigned)Wc);
            mbar_init(smem_u32(&sh->d_free[i]), CK_STORE_THREADS);
        }
        sh->abort_flag = 0u;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == CK_PRODUCER_WARP) {
        // ------------------------- producer: weight sub-tiles by TMA, ahead of the chain -----------
        if (lane == 0) {
            const int total = (L - 1) * P.nSub;
            const unsigned box_bytes = (unsigned)(Wc * P.R * sizeof(float));   // ragged edges are zero-filled
            int s = L, sub = 0, it = 0, st = 0;
            unsigned fill = 0;                       // how often the ring has been filled before
            for (; it < total; ++it) {
                if (fill > 0) {
                    ck_wait(smem_u32(&sh->empty[st]), (fill - 1) & 1u, P, sh);
                    if (sh->abort_flag) break;
                }
                const unsigned bar = smem_u32(&sh->full[st]);
                mbar_expect_tx(bar, box_bytes);
                tma_load_4d(smem_u32(ring + (size_t)st * P.stage_floats), &w_map, bar, col_base, 0, sub * P.RH, s - 1);
                if (++sub == P.nSub) { sub = 0; --s; }
                if (++st == P.stages) { st = 0; ++fill; }
            }
            // A CTA that gave up waiting may still have tiles on their way into its shared memory; it
            // must not exit under them.  Wait for the loads issued last, with a limit.
            if (sh->abort_flag) {
                const unsigned long long t0 = globaltimer_ns();
                for (int j = it > P.stages ? it - P.stages : 0; j < it; ++j) {
                    const unsigned bar = smem_u32(&sh->full[j % P.stages]);
                    const unsigned parity = (unsigned)((j / P.stages) & 1);
                    while (!mbar_try_wait(bar, parity) && globaltimer_ns() - t0 < 50000000ull) { }
                }
            }
        }
    } else if (warp >= CK_CHAIN_WARPS) {
        // ------------------------- store warps: rows [col_base, col_base + my_cols) of every gw^l ---
        const int st_tid = tid - CK_CHAIN_THREADS;
        const int n4 = N >> 2;
        for (int l = L; l >= 1; --l) {
            const int p = l & 1;
            const unsigned use = (unsigned)((L - l) >> 1);    // how often buffer p was used before
            const float4* a_prev = reinterpret_cast<const float4*>(P.a + (size_t)(l - 1) * N);
            float4 a4 = st_tid < n4 ? __ldg(a_prev + st_tid) : make_float4(0.f, 0.f, 0.f, 0.f);
            ck_wait(smem_u32(&sh->d_ready[p]), use & 1u, P, sh);
            // delta^l and gb^l (Eq. bp3) at this CTA's neurons, for the caller (every shard writes these)
            if (st_tid < my_cols && !(l == L && P.top_given)) {
                const float d = d_own[p * CK_MAX_WC + st_tid];
                P.delta[(size_t)(l - 1) * N + col_base + st_tid] = d;
                P.gb[(size_t)(l - 1) * N + col_base + st_tid] = d;
            }
            // layer-sharded form: another shard's layer is not stored (the waits and arrivals stay)
            const bool mine = P.shard_count == 1 || (L - l + P.depth_shift) % P.shard_count == P.shard_rank;
            if (mine) {
                const float* dr = d_own + p * CK_MAX_WC;
                float* out = P.gw + (size_t)(l - 1) * N * N + (size_t)col_base * N;
                const float* w_in = UPDATE ? P.w_sub + (size_t)(l - 1) * N * N + (size_t)col_base * N : nullptr;
                for (int c = st_tid; c < n4; c += CK_STORE_THREADS) {
                    const float4 av = a4;
                    if (c + CK_STORE_THREADS < n4) a4 = __ldg(a_prev + c + CK_STORE_THREADS);
                    if (UPDATE) {
                        for (int r0 = 0; r0 < my_cols; r0 += 4) {     // four loads of w in flight per thread
                            float4 wv[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (r0 + u < my_cols) wv[u] = __ldcg(reinterpret_cast<const float4*>(w_in + (size_t)(r0 + u) * N + 4 * c));
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                if (r0 + u < my_cols) {
                                    const float d = dr[r0 + u];
                                    st_stream4(out + (size_t)(r0 + u) * N + 4 * c,
                                               lf_sgd_apply4(P.eta, wv[u], make_float4(d * av.x, d * av.y, d * av.z, d * av.w)));
                                }
                            }
                        }
                    } else {
#pragma unroll 4
                        for (int r = 0; r < my_cols; ++r) {
                            const float d = dr[r];
                            st_stream4(out + (size_t)r * N + 4 * c, make_float4(d * av.x, d * av.y, d * av.z, d * av.w));
                        }
                    }
                }
            }
            mbar_arrive(smem_u32(&sh->d_free[p]));
        }
    } else {
        // ------------------------- chain warps ------------------------------------------------------
        const int WC4 = Wc >> 2;
        const int rpi = 32 / WC4;                   // tile rows a warp covers per iteration
        const bool active = lane < rpi * WC4;
        const int rsub = lane / WC4, c4 = lane - rsub * WC4;
        int pow2 = 1;
        while (pow2 < rpi) pow2 <<= 1;
        const int row_lo = warp * P.Rw, row_hi = min(P.R, row_lo + P.Rw);
        const bool finisher = tid < Wc;
        const int my_col = col_base + tid;
        const bool col_ok = finisher && my_col < N;

        // ---- Eq. bp1 at my columns: rows of gw^L for the store warps; delta^L and gb^L (Eq. bp3)
        if (finisher) {
            float d = 0.f;
            if (col_ok) {
                d = ck_top_delta(P, my_col);
            }
            d_own[(L & 1) * CK_MAX_WC + tid] = d;
            mbar_arrive(smem_u32(&sh->d_ready[L & 1]));
        }
        float a_mine = (col_ok && L >= 2) ? P.a[(size_t)(L - 1) * N + my_col] : 0.f;

        int st = 0;
        unsigned full_phase = 0;
        const int n_items = P.nSub * ((P.Rw + 31) >> 5);
        CkPoll q;
        q.sub = 0; q.piece = 0;
        for (int s = L; s >= 2; --s) {
            CK_STAMP(0);
            const float a_mine_next = (col_ok && s >= 3) ? P.a[(size_t)(s - 2) * N + my_col] : 0.f;
            const unsigned long long* slots = P.xch + (size_t)(s - 1) * N;
            q.sub = 0; q.piece = 0;
            // delta^s of this warp's rows: Eq. bp1 at the top, polled below it
            if (s == L) {
                for (int i0 = 0; i0 < n_items; i0 += CK_POLL_BATCH) {
                    ck_poll_setup(q, P.R, P.Rw, P.nSub, P.N, warp, lane);
#pragma unroll
                    for (int u = 0; u < CK_POLL_BATCH; ++u)
                        if (q.valid[u]) d_sm[q.row[u]] = q.pend[u] ? ck_top_delta(P, q.row[u]) : 0.f;
                }
            } else {
                for (int i0 = 0; i0 < n_items; i0 += CK_POLL_BATCH) {
                    ck_poll_setup(q, P.R, P.Rw, P.nSub, P.N, warp, lane);
                    ck_poll_issue(q, slots);
                    ck_poll_collect(q, P, sh, slots, d_sm);
                }
            }
            __syncwarp();
            CK_STAMP(1);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int sub = 0; sub < P.nSub; ++sub) {
                ck_wait(smem_u32(&sh->full[st]), full_phase, P, sh);
                const float4* tile = reinterpret_cast<const float4*>(ring + (size_t)st * P.stage_floats);
                const float* dsub = d_sm + sub * P.R;
                if (active) {
#pragma unroll 4
                    for (int r = row_lo + rsub; r < row_hi; r += rpi) {
                        const float4 wv = tile[r * WC4 + c4];
                        const float d = dsub[r];
                        acc.x = fmaf(wv.x, d, acc.x);
                        acc.y = fmaf(wv.y, d, acc.y);
                        acc.z = fmaf(wv.z, d, acc.z);
                        acc.w = fmaf(wv.w, d, acc.w);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh->empty[st]));
                if (++st == P.stages) { st = 0; full_phase ^= 1u; }
            }
            CK_STAMP(2);
            // the warp's rows: a fixed tree over the lanes that hold the same four columns
            {
                int cnt = rpi;
                for (int stp = pow2 >> 1; stp >= 1; stp >>= 1) {
                    const float4 o = make_float4(__shfl_down_sync(0xffffffffu, acc.x, stp * WC4),
                                                 __shfl_down_sync(0xffffffffu, acc.y, stp * WC4),
                                                 __shfl_down_sync(0xffffffffu, acc.z, stp * WC4),
                                                 __shfl_down_sync(0xffffffffu, acc.w, stp * WC4));
                    if (rsub < stp && rsub + stp < cnt) { acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
                    if (cnt > stp) cnt = stp;
                }
            }
            const int p = s & 1;
            float4* red_p = red + p * CK_CHAIN_WARPS * 32;
            if (lane < WC4) red_p[warp * 32 + lane] = acc;
            bar_sync(1, CK_CHAIN_THREADS);
            CK_STAMP(3);
            float d = 0.f;
            if (finisher) {
                // the eight warps' sums of my column, added in warp order
                const float* rp = reinterpret_cast<const float*>(red_p);
                float part[CK_CHAIN_WARPS];
#pragma unroll
                for (int wq = 0; wq < CK_CHAIN_WARPS; ++wq) part[wq] = rp[wq * 128 + tid];
                float v = part[0];
#pragma unroll
                for (int wq = 1; wq < CK_CHAIN_WARPS; ++wq) v += part[wq];
                if (col_ok) {
                    d = v * lf_act_prime(a_mine, P.act);                                   // Eq. bp2
                    if (!(P.withhold && blockIdx.x == 0)) st_slot(P.xch + (size_t)(s - 2) * N + my_col, d, P.epoch);
                }
            }
            CK_STAMP(4);
            if (finisher) {
                // hand delta^{s-1} of my column to the store warps: it scales row my_col of gw^{s-1},
                // and they also write it to delta and gb (Eq. bp3), which nothing on the chain reads
                const int pn = (s - 1) & 1;
                const unsigned used = (unsigned)((L - (s - 1)) >> 1);   // earlier uses of buffer pn
                if (used > 0) ck_wait(smem_u32(&sh->d_free[pn]), (used - 1) & 1u, P, sh);
                d_own[pn * CK_MAX_WC + tid] = d;
                mbar_arrive(smem_u32(&sh->d_ready[pn]));
            }
            a_mine = a_mine_next;
        }
    }
    __syncthreads();
}

// ---- the same pass for layers of different widths ------------------------------------------------
// Step s reads w^s (n_s rows, n_{s-1} columns) and produces delta^{s-1}; CTA q owns the columns
// [q * Wc_s, (q+1) * Wc_s) of that matrix, with Wc_s following the layer, so every layer keeps all
// CTAs busy whatever its shape.  Everything a step needs is one entry of a table (copied to shared
// memory when the kernel starts) and one tensor map per layer.  The uniform kernel above is this
// one with every entry equal; it stays a kernel of its own because its constants come for free.
constexpr int CK_TAB_MAX = 64;     // layers the table holds
struct CkLayer {
    int rows, cols;        // n_s, n_{s-1}: the shape of w^s
    int Wc;                // columns of w^s per CTA (= neurons of layer s-1 a CTA finishes)
    int RH, R, nSub, Rw;   // TMA box (RL x RH rows) and the warps' shares of it
    unsigned box_bytes;
    unsigned off_w_lo, off_w_hi;   // start of w^s / gw^s (floats, 64 bits)
    int off_rows;          // start of delta^s in delta / gb / the exchange slots (B = 1: neurons before layer s)
    int off_cols;          // start of delta^{s-1} there
    int off_a_cols;        // start of a^{s-1} in a
    int Wc_rows;           // neurons of layer s a CTA finishes (its rows of gw^s)
    int pad0, pad1;
};
static_assert(sizeof(CkLayer) == 64, "one table entry is 64 bytes");

template <bool UPDATE>
__global__ void __launch_bounds__(CK_THREADS, 1)
k_backward_columns_widths(const CUtensorMap* __restrict__ maps, const CkLayer* __restrict__ table, const CkParams P)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    float* ring = reinterpret_cast<float*>(smem_raw);                                // stages x stage_floats
    float* d_sm = ring + (size_t)P.stages * P.stage_floats;                          // [max nSub * R]
    float4* red = reinterpret_cast<float4*>(d_sm + (((size_t)P.nSub * P.R + 3) & ~(size_t)3));   // [2][8 warps][32]
    float* d_own = reinterpret_cast<float*>(red + 2 * CK_CHAIN_WARPS * 32);          // [2][CK_MAX_WC]
    CkLayer* tab = reinterpret_cast<CkLayer*>(d_own + 2 * CK_MAX_WC);                // [L + 1], entry s for step s
    CkShared* sh = reinterpret_cast<CkShared*>(tab + CK_TAB_MAX + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = P.L;
    for (int i = tid; i < (L + 1) * (int)(sizeof(CkLayer) / 16); i += CK_THREADS)
        reinterpret_cast<float4*>(tab)[i] = reinterpret_cast<const float4*>(table)[i];
    if (tid == 0) {
        for (int i = 0; i < P.stages; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->empty[i]), CK_CHAIN_WARPS);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh->d_ready[i]), CK_MAX_WC);     // the first 128 chain threads, finishing or not
            mbar_init(smem_u32(&sh->d_free[i]), CK_STORE_THREADS);
        }
        sh->abort_flag = 0u;
        mbar_fence_init();
    }
    __syncthreads();
    // entry s (2 <= s <= L) describes step s; entry 1 only the top of the table's use by the stores
    // (rows of gw^1); Wc_rows of entry L is the split of the top layer.

    if (warp == CK_PRODUCER_WARP) {
        if (lane == 0) {
            int it = 0, st = 0;
            unsigned fill = 0;
            for (int s = L; s >= 2 && !sh->abort_flag; --s) {
                const CkLayer ly = tab[s];
                const int col_base = blockIdx.x * ly.Wc;
                for (int sub = 0; sub < ly.nSub; ++sub, ++it) {
                    if (fill > 0) {
                        ck_wait(smem_u32(&sh->empty[st]), (fill - 1) & 1u, P, sh);
                        if (sh->abort_flag) break;
                    }
                    const unsigned bar = smem_u32(&sh->full[st]);
                    mbar_expect_tx(bar, ly.box_bytes);
                    // (a CTA whose columns lie beyond the matrix still loads: the box is all fill)
                    tma_load_3d(smem_u32(ring + (size_t)st * P.stage_floats), maps + (s - 1), bar, col_base, 0, sub * ly.RH);
                    if (++st == P.stages) { st = 0; ++fill; }
                }
            }
            if (sh->abort_flag) {
                const unsigned long long t0 = globaltimer_ns();
                for (int j = it > P.stages ? it - P.stages : 0; j < it; ++j) {
                    const unsigned bar = smem_u32(&sh->full[j % P.stages]);
                    const unsigned parity = (unsigned)((j / P.stages) & 1);
                    while (!mbar_try_wait(bar, parity) && globaltimer_ns() - t0 < 50000000ull) { }
                }
            }
        }
    } else if (warp >= CK_CHAIN_WARPS) {
        // ------------------------- store warps: this CTA's rows of every gw^l -----------------------
        const int st_tid = tid - CK_CHAIN_THREADS;
        for (int l = L; l >= 1; --l) {
            const CkLayer ly = tab[l];                       // w^l: rows = n_l, cols = n_{l-1}
            const int p = l & 1;
            const unsigned use = (unsigned)((L - l) >> 1);
            const int n4 = ly.cols >> 2;
            const int row_base = blockIdx.x * ly.Wc_rows;
            const int my_rows = min(ly.Wc_rows, ly.rows - row_base);        // <= 0: none of this layer
            const float4* a_prev = reinterpret_cast<const float4*>(P.a + ly.off_a_cols);
            float4 a4 = st_tid < n4 ? __ldg(a_prev + st_tid) : make_float4(0.f, 0.f, 0.f, 0.f);
            ck_wait(smem_u32(&sh->d_ready[p]), use & 1u, P, sh);
            if (st_tid < my_rows && !(l == L && P.top_given)) {
                const float d = d_own[p * CK_MAX_WC + st_tid];
                P.delta[ly.off_rows + row_base + st_tid] = d;
                P.gb[ly.off_rows + row_base + st_tid] = d;                  // Eq. bp3
            }
            const bool mine = P.shard_count == 1 || (L - l + P.depth_shift) % P.shard_count == P.shard_rank;
            if (mine && my_rows > 0) {
                const float* dr = d_own + p * CK_MAX_WC;
                const size_t off_w = ((size_t)ly.off_w_hi << 32) | ly.off_w_lo;
                float* out = P.gw + off_w + (size_t)row_base * ly.cols;
                const float* w_in = UPDATE ? P.w_sub + off_w + (size_t)row_base * ly.cols : nullptr;
                for (int c = st_tid; c < n4; c += CK_STORE_THREADS) {
                    const float4 av = a4;
                    if (c + CK_STORE_THREADS < n4) a4 = __ldg(a_prev + c + CK_STORE_THREADS);
                    if (UPDATE) {
                        for (int r0 = 0; r0 < my_rows; r0 += 4) {
                            float4 wv[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (r0 + u < my_rows) wv[u] = __ldcg(reinterpret_cast<const float4*>(w_in + (size_t)(r0 + u) * ly.cols + 4 * c));
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                if (r0 + u < my_rows) {
                                    const float d = dr[r0 + u];
                                    st_stream4(out + (size_t)(r0 + u) * ly.cols + 4 * c,
                                               lf_sgd_apply4(P.eta, wv[u], make_float4(d * av.x, d * av.y, d * av.z, d * av.w)));
                                }
                            }
                        }
                    } else {
#pragma unroll 4
                        for (int r = 0; r < my_rows; ++r) {
                            const float d = dr[r];
                            st_stream4(out + (size_t)r * ly.cols + 4 * c, make_float4(d * av.x, d * av.y, d * av.z, d * av.w));
                        }
                    }
                }
            }
            mbar_arrive(smem_u32(&sh->d_free[p]));
        }
    } else {
        // ------------------------- chain warps ------------------------------------------------------
        const bool hands_over = tid < CK_MAX_WC;     // these threads fill d_own (with 0 where they finish nothing)
        // ---- Eq. bp1 at the top layer's neurons of this CTA
        {
            const CkLayer top = tab[L];
            const int r = blockIdx.x * top.Wc_rows + tid;
            if (hands_over) {
                float d = 0.f;
                if (tid < top.Wc_rows && r < top.rows)
                    d = ck_top_delta_at(P, P.a + top.off_a_cols + top.cols, P.delta + top.off_rows, r);
                d_own[(L & 1) * CK_MAX_WC + tid] = d;
                mbar_arrive(smem_u32(&sh->d_ready[L & 1]));
            }
        }
        int st = 0;
        unsigned full_phase = 0;
        CkPoll q;
        for (int s = L; s >= 2; --s) {
            const CkLayer ly = tab[s];
            const int Wc = ly.Wc, WC4 = Wc >> 2, rpi = 32 / WC4;
            const bool active = lane < rpi * WC4;
            const int rsub = lane / WC4, c4 = lane - rsub * WC4;
            int pow2 = 1;
            while (pow2 < rpi) pow2 <<= 1;
            const int row_lo = warp * ly.Rw, row_hi = min(ly.R, row_lo + ly.Rw);
            const int my_col = blockIdx.x * Wc + tid;
            const bool col_ok = tid < Wc && my_col < ly.cols;
            const float a_mine = col_ok ? P.a[ly.off_a_cols + my_col] : 0.f;
            const unsigned long long* slots = P.xch + ly.off_rows;
            const int n_items = ly.nSub * ((ly.Rw + 31) >> 5);
            q.sub = 0; q.piece = 0;
            if (s == L) {
                const CkLayer top = ly;
                for (int i0 = 0; i0 < n_items; i0 += CK_POLL_BATCH) {
                    ck_poll_setup(q, ly.R, ly.Rw, ly.nSub, ly.rows, warp, lane);
#pragma unroll
                    for (int u = 0; u < CK_POLL_BATCH; ++u)
                        if (q.valid[u])
                            d_sm[q.row[u]] = q.pend[u] ? ck_top_delta_at(P, P.a + top.off_a_cols + top.cols, P.delta + top.off_rows, q.row[u]) : 0.f;
                }
            } else {
                for (int i0 = 0; i0 < n_items; i0 += CK_POLL_BATCH) {
                    ck_poll_setup(q, ly.R, ly.Rw, ly.nSub, ly.rows, warp, lane);
                    ck_poll_issue(q, slots);
                    ck_poll_collect(q, P, sh, slots, d_sm);
                }
            }
            __syncwarp();
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int sub = 0; sub < ly.nSub; ++sub) {
                ck_wait(smem_u32(&sh->full[st]), full_phase, P, sh);
                const float4* tile = reinterpret_cast<const float4*>(ring + (size_t)st * P.stage_floats);
                const float* dsub = d_sm + sub * ly.R;
                if (active) {
#pragma unroll 4
                    for (int r = row_lo + rsub; r < row_hi; r += rpi) {
                        const float4 wv = tile[r * WC4 + c4];
                        const float d = dsub[r];
                        acc.x = fmaf(wv.x, d, acc.x);
                        acc.y = fmaf(wv.y, d, acc.y);
                        acc.z = fmaf(wv.z, d, acc.z);
                        acc.w = fmaf(wv.w, d, acc.w);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh->empty[st]));
                if (++st == P.stages) { st = 0; full_phase ^= 1u; }
            }
            {
                int cnt = rpi;
                for (int stp = pow2 >> 1; stp >= 1; stp >>= 1) {
                    const float4 o = make_float4(__shfl_down_sync(0xffffffffu, acc.x, stp * WC4),
                                                 __shfl_down_sync(0xffffffffu, acc.y, stp * WC4),
                                                 __shfl_down_sync(0xffffffffu, acc.z, stp * WC4),
                                                 __shfl_down_sync(0xffffffffu, acc.w, stp * WC4));
                    if (rsub < stp && rsub + stp < cnt) { acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
                    if (cnt > stp) cnt = stp;
                }
            }
            float4* red_p = red + (s & 1) * CK_CHAIN_WARPS * 32;
            if (lane < WC4) red_p[warp * 32 + lane] = acc;
            bar_sync(1, CK_CHAIN_THREADS);
            float d = 0.f;
            if (tid < Wc) {
                const float* rp = reinterpret_cast<const float*>(red_p);
                float part[CK_CHAIN_WARPS];
#pragma unroll
                for (int wq = 0; wq < CK_CHAIN_WARPS; ++wq) part[wq] = rp[wq * 128 + tid];
                float v = part[0];
#pragma unroll
                for (int wq = 1; wq < CK_CHAIN_WARPS; ++wq) v += part[wq];
                if (col_ok) {
                    d = v * lf_act_prime(a_mine, P.act);                                   // Eq. bp2
                    if (!(P.withhold && blockIdx.x == 0)) st_slot(P.xch + ly.off_cols + my_col, d, P.epoch);
                }
            }
            if (hands_over) {
                const int pn = (s - 1) & 1;
                const unsigned used = (unsigned)((L - (s - 1)) >> 1);
                if (used > 0) ck_wait(smem_u32(&sh->d_free[pn]), (used - 1) & 1u, P, sh);
                d_own[pn * CK_MAX_WC + tid] = d;
                mbar_arrive(smem_u32(&sh->d_ready[pn]));
            }
        }
    }
    __syncthreads();
}

struct CkPlan {
    bool ok;
    int Q, Wc, RL, RH, R, nSub, Rw, stages, stage_floats;
    size_t smem_bytes;
};

typedef CUresult (*ck_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

ck_encode_fn ck_get_encode_fn()
{
    static ck_encode_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<ck_encode_fn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// CTAs of this kernel the device keeps resident at once (one per multiprocessor at this
// shared-memory size); 0 if the kernel cannot run here.
int ck_max_ctas(const lf_ctx* c)
{
    static int cached_dev = -1, cached = 0;
    if (cached_dev == c->device) return cached;
    int per_sm = 0;
    int per_sm_upd = 0;
    if (cudaFuncSetAttribute(k_backward_columns<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)CK_SMEM_LIMIT) != cudaSuccess ||
        cudaFuncSetAttribute(k_backward_columns<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)CK_SMEM_LIMIT) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_backward_columns<false>, CK_THREADS, CK_SMEM_LIMIT) !=
            cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_upd, k_backward_columns<true>, CK_THREADS, CK_SMEM_LIMIT) !=
            cudaSuccess)
        per_sm = 0;
    if (per_sm_upd < per_sm) per_sm = per_sm_upd;
    cudaGetLastError();
    int coop = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
    cached_dev = c->device;
    cached = coop ? (per_sm > 0 ? c->sm_count : 0) : 0;
    return cached;
}

CkPlan ck_make_plan(const lf_ctx* c)
{
    CkPlan p = {};
    const int N = c->pk_N;
    if (c->B != 1 || N <= 0 || N > CK_MAX_N || c->pk_L < 1) return p;
    if ((size_t)c->smem_optin < CK_SMEM_LIMIT || !ck_get_encode_fn()) return p;
    const int max_ctas = ck_max_ctas(c);
    if (max_ctas < 1) return p;
    p.Wc = 4 * ((N + 4 * max_ctas - 1) / (4 * max_ctas));
    if (p.Wc < CK_MIN_WC && N >= CK_MIN_WC) p.Wc = CK_MIN_WC;   // rows of at least 32 bytes per TMA box row
    if (p.Wc > CK_MAX_WC) return p;
    p.Q = (N + p.Wc - 1) / p.Wc;
    // TMA box: RL rows, the largest even divisor of N up to 256 that fits a stage (even: delta is
    // polled in pairs of rows), times RH blocks of RL rows
    p.RL = 2;
    for (int d = CK_STAGE_FLOATS / p.Wc < 256 ? CK_STAGE_FLOATS / p.Wc : 256; d >= 1; --d)
        if (N % d == 0 && d % 2 == 0) { p.RL = d; break; }
    p.RH = CK_STAGE_FLOATS / (p.Wc * p.RL);
    if (p.RH > N / p.RL) p.RH = N / p.RL;
    if (p.RH > 256) p.RH = 256;
    if (p.RH < 1) return p;
    p.R = p.RL * p.RH;
    p.nSub = (N / p.RL + p.RH - 1) / p.RH;
    p.Rw = 2 * ((p.R + 2 * CK_CHAIN_WARPS - 1) / (2 * CK_CHAIN_WARPS));
    p.stage_floats = (p.R * p.Wc + 31) & ~31;      // 128-byte multiples
    const size_t fixed = (((size_t)p.nSub * p.R + 3) & ~(size_t)3) * 4 + 2 * CK_CHAIN_WARPS * 32 * 16 + 2 * CK_MAX_WC * 4 + sizeof(CkShared) + 16;
    if (fixed + 2 * (size_t)p.stage_floats * 4 > CK_SMEM_LIMIT) return p;
    size_t st = (CK_SMEM_LIMIT - fixed) / ((size_t)p.stage_floats * 4);
    if (st > CK_MAX_STAGES) st = CK_MAX_STAGES;
    p.stages = (int)st;
    p.smem_bytes = fixed + (size_t)p.stages * p.stage_floats * 4;
    p.ok = true;
    return p;
}

}  // namespace

bool lf_columns_supported(const lf_ctx* c) { return ck_make_plan(c).ok; }

// The launch covers the pk_L layers of width pk_N that w, a, delta, gw, gb point at (the whole
// network, or the run of equal-width hidden layers: top_given, depth_shift as in the cluster kernel).
int lf_backward_columns(lf_ctx* c, const float* w, const float* a, const float* y, float* delta, float* gw,
                        float* gb, const float* w_sub, int top_given, int depth_shift)
{
    const int L_run = c->pk_L, N_run = c->pk_N;
    const CkPlan pl = ck_make_plan(c);
    if (!pl.ok) return LF_ERESOURCE;
    // tensor map over w as [L][N / RL][RL][N]; box = Wc columns x RL rows x RH row blocks x 1 layer
    if (!c->ck_map_valid || c->ck_map_ptr != w || c->ck_map_wc != pl.Wc) {
        CUtensorMap* m = reinterpret_cast<CUtensorMap*>(c->ck_map_storage);
        cuuint64_t dims[4] = {(cuuint64_t)N_run, (cuuint64_t)pl.RL, (cuuint64_t)(N_run / pl.RL), (cuuint64_t)L_run};
        cuuint64_t strides[3] = {(cuuint64_t)N_run * 4, (cuuint64_t)N_run * pl.RL * 4, (cuuint64_t)N_run * N_run * 4};
        cuuint32_t box[4] = {(cuuint32_t)pl.Wc, (cuuint32_t)pl.RL, (cuuint32_t)pl.RH, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = ck_get_encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(w), dims, strides,
                                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            c->last_cuda_error = (int)r;
            return LF_ECUDA;
        }
        c->ck_map_valid = true; c->ck_map_ptr = w; c->ck_map_wc = pl.Wc;
    }
    c->epoch += 1;
    if (c->epoch == 0) c->epoch = 1;

    CkParams P = {};
    P.L = L_run; P.N = N_run; P.Q = pl.Q; P.Wc = pl.Wc; P.RL = pl.RL; P.RH = pl.RH; P.R = pl.R;
    P.nSub = pl.nSub; P.Rw = pl.Rw; P.stages = pl.stages; P.stage_floats = pl.stage_floats;
    P.top_given = top_given; P.depth_shift = depth_shift;
    P.shard_rank = c->shard_rank; P.shard_count = c->shard_count > 1 ? c->shard_count : 1;
    P.withhold = c->withhold == 1 ? 1 : 0; P.cost = c->opt_cost; P.act = c->opt_act;
    P.epoch = c->epoch;
    P.budget_ns = (unsigned long long)c->wait_budget_us * 1000ull;
    P.a = a; P.y = y; P.delta = delta; P.gw = gw; P.gb = gb;
    P.w_sub = c->sgd_on ? w_sub : nullptr; P.eta = c->sgd_eta;
    P.xch = reinterpret_cast<unsigned long long*>(c->sync_words);
    P.status = c->status_dev;
#ifdef LF_CK_TRACE
    if (!c->trace_dev) cudaMalloc(&c->trace_dev, (size_t)2 * c->L * 16 * sizeof(unsigned long long));
    cudaMemsetAsync(c->trace_dev, 0, (size_t)2 * c->L * 16 * sizeof(unsigned long long), c->stream);
    P.trace = c->trace_dev;
#endif

    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_columns<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)CK_SMEM_LIMIT));
    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_columns<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)CK_SMEM_LIMIT));
    // the CTAs wait for each other: a cooperative launch runs only if all of them are resident at once
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    cfg.gridDim = dim3(pl.Q);
    cfg.blockDim = dim3(CK_THREADS);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = c->stream;
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const CUtensorMap* mp = reinterpret_cast<const CUtensorMap*>(c->ck_map_storage);
    if (P.w_sub)
        LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_columns<true>, *mp, P));
    else
        LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_columns<false>, *mp, P));
    c->stats.launches_backward = 1;
    c->stats.chain_ctas = pl.Q;
    c->stats.worker_ctas = 0;
    return LF_OK;
}


// ---- layers of different widths: plan, table, tensor maps, launch ----------------------------------
namespace {

struct CkWidthsPlan {
    bool ok;
    int Q, stages, stage_floats, d_floats;
    size_t smem_bytes;
};

// Fills `tab` (L + 1 entries, entry 0 unused) and the box shapes; returns the launch plan.
CkWidthsPlan ck_plan_widths(const lf_ctx* c, CkLayer* tab, int* rl_out)
{
    CkWidthsPlan p = {};
    const int L = c->L;
    if (c->B != 1 || L < 1 || L > CK_TAB_MAX) return p;
    if ((size_t)c->smem_optin < CK_SMEM_LIMIT || !ck_get_encode_fn()) return p;
    const int max_ctas = ck_max_ctas(c);
    if (max_ctas < 1) return p;
    auto split = [&](int n) {                       // neurons of a layer per CTA
        int wc = 4 * ((n + 4 * max_ctas - 1) / (4 * max_ctas));
        if (wc < CK_MIN_WC && n >= CK_MIN_WC) wc = CK_MIN_WC;
        return wc;
    };
    int q_needed = 1;
    for (int l = 1; l <= L; ++l) {
        CkLayer& e = tab[l];
        e = CkLayer{};
        e.rows = c->width[l]; e.cols = c->width[l - 1];
        if (e.rows > CK_MAX_N || e.cols > CK_MAX_N) return p;
        e.Wc_rows = split(e.rows);
        e.Wc = split(e.cols);                       // (entry 1: not used, the chain ends at step 2)
        if (e.Wc_rows > CK_MAX_WC || e.Wc > CK_MAX_WC) return p;
        const size_t ow = c->off_w[l - 1];
        e.off_w_lo = (unsigned)(ow & 0xffffffffu); e.off_w_hi = (unsigned)(ow >> 32);
        if (c->off_h[L] > 0x7fffffffu || c->off_a[L + 1] > 0x7fffffffu) return p;
        e.off_rows = (int)c->off_h[l - 1];
        e.off_cols = l >= 2 ? (int)c->off_h[l - 2] : 0;
        e.off_a_cols = (int)c->off_a[l - 1];
        const int q_rows = (e.rows + e.Wc_rows - 1) / e.Wc_rows;
        if (q_rows > q_needed) q_needed = q_rows;
        if (l >= 2) {
            int RL = 2;
            for (int d = CK_STAGE_FLOATS / e.Wc < 256 ? CK_STAGE_FLOATS / e.Wc : 256; d >= 1; --d)
                if (e.rows % d == 0 && d % 2 == 0) { RL = d; break; }
            rl_out[l] = RL;
            e.RH = CK_STAGE_FLOATS / (e.Wc * RL);
            if (e.RH > e.rows / RL) e.RH = e.rows / RL;
            if (e.RH > 256) e.RH = 256;
            if (e.RH < 1) return p;
            e.R = RL * e.RH;
            e.nSub = (e.rows / RL + e.RH - 1) / e.RH;
            e.Rw = 2 * ((e.R + 2 * CK_CHAIN_WARPS - 1) / (2 * CK_CHAIN_WARPS));
            e.box_bytes = (unsigned)(e.Wc * e.R * sizeof(float));
            const int sf = (e.R * e.Wc + 31) & ~31;
            if (sf > p.stage_floats) p.stage_floats = sf;
            if (e.nSub * e.R > p.d_floats) p.d_floats = e.nSub * e.R;
            const int q_cols = (e.cols + e.Wc - 1) / e.Wc;
            if (q_cols > q_needed) q_needed = q_cols;
        }
    }
    // a CTA finishes the same neurons of layer l whether they are columns of w^{l+1} or rows of gw^l
    for (int l = 1; l < L; ++l)
        if (tab[l].Wc_rows != tab[l + 1].Wc) return p;
    if (p.stage_floats == 0) { p.stage_floats = 32; p.d_floats = 4; }      // L == 1: no chain step
    p.Q = q_needed;
    if (p.Q > max_ctas) return p;
    const size_t fixed = (((size_t)p.d_floats + 3) & ~(size_t)3) * 4 + 2 * CK_CHAIN_WARPS * 32 * 16 + 2 * CK_MAX_WC * 4 +
                         (CK_TAB_MAX + 1) * sizeof(CkLayer) + sizeof(CkShared) + 16;
    if (fixed + 2 * (size_t)p.stage_floats * 4 > CK_SMEM_LIMIT) return p;
    size_t st = (CK_SMEM_LIMIT - fixed) / ((size_t)p.stage_floats * 4);
    if (st > CK_MAX_STAGES) st = CK_MAX_STAGES;
    p.stages = (int)st;
    p.smem_bytes = fixed + (size_t)p.stages * p.stage_floats * 4;
    p.ok = true;
    return p;
}

}  // namespace

bool lf_columns_widths_supported(const lf_ctx* c)
{
    if (c->uniform) return false;
    CkLayer tab[CK_TAB_MAX + 1];
    int rl[CK_TAB_MAX + 1];
    return ck_plan_widths(c, tab, rl).ok;
}

void lf_columns_release(lf_ctx* c)
{
    if (c->ckw_dev) cudaFree(c->ckw_dev);
    c->ckw_dev = nullptr;
}

// One launch over all L layers of a context whose layers differ in width (B = 1).
int lf_backward_columns_widths(lf_ctx* c, const float* w, const float* a, const float* y, float* delta, float* gw,
                               float* gb, const float* w_sub)
{
    const int L = c->L;
    CkLayer tab[CK_TAB_MAX + 1];
    int rl[CK_TAB_MAX + 1] = {};
    const CkWidthsPlan pl = ck_plan_widths(c, tab, rl);
    if (!pl.ok) return LF_ERESOURCE;
    // device copy of the table and of one tensor map per layer, rebuilt when the weights move
    const size_t maps_bytes = (size_t)L * sizeof(CUtensorMap), tab_bytes = (size_t)(L + 1) * sizeof(CkLayer);
    if (!c->ckw_dev) {
        cudaError_t e = cudaMalloc(&c->ckw_dev, maps_bytes + tab_bytes);
        if (e != cudaSuccess) {
            c->ckw_dev = nullptr;
            c->last_cuda_error = (int)e;
            cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? LF_ENOMEM : LF_ECUDA;
        }
        c->stats.workspace_bytes += (long long)(maps_bytes + tab_bytes);
        c->ckw_ptr = nullptr;
    }
    if (c->ckw_ptr != w) {
        alignas(64) CUtensorMap maps[CK_TAB_MAX];
        memset(maps, 0, sizeof(maps));
        for (int s = 2; s <= L; ++s) {        // w^s as [rows / RL][RL][cols]; box = Wc columns x RL rows x RH row blocks
            const CkLayer& e = tab[s];
            const size_t ow = ((size_t)e.off_w_hi << 32) | e.off_w_lo;
            cuuint64_t dims[3] = {(cuuint64_t)e.cols, (cuuint64_t)rl[s], (cuuint64_t)(e.rows / rl[s])};
            cuuint64_t strides[2] = {(cuuint64_t)e.cols * 4, (cuuint64_t)e.cols * rl[s] * 4};
            cuuint32_t box[3] = {(cuuint32_t)e.Wc, (cuuint32_t)rl[s], (cuuint32_t)e.RH};
            cuuint32_t estr[3] = {1, 1, 1};
            CUresult r = ck_get_encode_fn()(&maps[s - 1], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(w + ow), dims,
                                            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) {
                c->last_cuda_error = (int)r;
                return LF_ECUDA;
            }
        }
        // (pageable host memory: the copies are staged by the runtime before the calls return)
        LF_CUDA_TRY(c, cudaMemcpyAsync(c->ckw_dev, maps, maps_bytes, cudaMemcpyHostToDevice, c->stream));
        LF_CUDA_TRY(c, cudaMemcpyAsync(static_cast<unsigned char*>(c->ckw_dev) + maps_bytes, tab, tab_bytes,
                                       cudaMemcpyHostToDevice, c->stream));
        c->ckw_ptr = w;
    }
    c->epoch += 1;
    if (c->epoch == 0) c->epoch = 1;

    CkParams P = {};
    P.L = L; P.N = c->N; P.Q = pl.Q;
    P.R = pl.d_floats; P.nSub = 1;                 // (only the size of the delta buffer is taken from these)
    P.stages = pl.stages; P.stage_floats = pl.stage_floats;
    P.top_given = 0; P.depth_shift = 0;
    P.shard_rank = c->shard_rank; P.shard_count = c->shard_count > 1 ? c->shard_count : 1;
    P.withhold = c->withhold == 1 ? 1 : 0; P.cost = c->opt_cost; P.act = c->opt_act;
    P.epoch = c->epoch;
    P.budget_ns = (unsigned long long)c->wait_budget_us * 1000ull;
    P.a = a; P.y = y; P.delta = delta; P.gw = gw; P.gb = gb;
    P.w_sub = c->sgd_on ? w_sub : nullptr; P.eta = c->sgd_eta;
    P.xch = reinterpret_cast<unsigned long long*>(c->sync_words);
    P.status = c->status_dev;

    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_columns_widths<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)CK_SMEM_LIMIT));
    LF_CUDA_TRY(c, cudaFuncSetAttribute(k_backward_columns_widths<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)CK_SMEM_LIMIT));
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    cfg.gridDim = dim3(pl.Q);
    cfg.blockDim = dim3(CK_THREADS);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = c->stream;
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const CUtensorMap* maps_dev = static_cast<const CUtensorMap*>(c->ckw_dev);
    const CkLayer* tab_dev = reinterpret_cast<const CkLayer*>(static_cast<unsigned char*>(c->ckw_dev) + maps_bytes);
    if (P.w_sub)
        LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_columns_widths<true>, maps_dev, tab_dev, P));
    else
        LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_backward_columns_widths<false>, maps_dev, tab_dev, P));
    c->stats.launches_backward = 1;
    c->stats.chain_ctas = pl.Q;
    c->stats.worker_ctas = 0;
    c->stats.fused_tiling = LF_FUSED_TILING_COLUMNS;
    return LF_OK;
}
