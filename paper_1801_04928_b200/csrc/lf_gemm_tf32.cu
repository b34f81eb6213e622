// Mini-batch weight gradient (Eq. bp4 summed over the B samples) on the 5th-generation tensor
// cores:  G[j][k] = sum_b D[b][j] * A[b][k],  D = delta^l [B][N], A = a^{l-1} [B][N], G = gw^l.
//
// An N x N x B contraction whose contraction index b is the SLOW index of both operands, i.e.
// both are "MN-major".  One persistent CTA per SM works through 128 x 256 output tiles:
//   warp 0     TMA producer: 32 samples of D (128 columns) and of A (256 columns) per stage, as
//              boxes of 32 floats x 32 rows in the 128-byte swizzle with 32-byte atoms -- the one
//              shared-memory layout the tensor core accepts for MN-major 32-bit operands -- so
//              the [B][N] arrays are used as they are, with no repacking;
//   warp 1     issues tcgen05.mma kind::tf32 (M = 128, N = 256, K = 8 per instruction), fp32
//              accumulators in tensor memory, two accumulator buffers of 256 columns;
//   warps 2-5  epilogue: tcgen05.ld the finished accumulator (one 32-lane quadrant per warp)
//              and store it to gw while the next tile is being multiplied.
// The tensor core takes the upper 19 bits of each fp32 operand (TF32); accumulation is fp32.
// Ragged edges: TMA fills out-of-range columns / samples with zeros, stores are bounds-checked.
// Every mbarrier wait is bounded; on expiry the status word is raised and the CTA drains out.
#include <cuda.h>

#include "lf_internal.h"
#include "lf_ptx.cuh"

// Debug builds (-DLF_TG_TRACE): the leader CTA of pair 0 of the two-SM kernel stamps its SM clock per
// tile (words 16 t + slot) and once per launch (words 8 .. 11 of tile 0); the release library carries
// none of this.
#ifdef LF_TG_TRACE
constexpr int TG_TRACE_TILES = 32;
__device__ long long tg_trace[TG_TRACE_TILES * 16];
extern "C" int lf_debug_read_gw_pair_trace(long long* out)
{
    if (!out) return LF_ENULL;
    cudaDeviceSynchronize();
    return cudaMemcpyFromSymbol(out, tg_trace, sizeof(tg_trace)) == cudaSuccess ? LF_OK : LF_ECUDA;
}
// per tile: 0 issuer has the accumulator, 1 first stage's operands seen, 2 all products and commits issued,
// 3 an epilogue warp sees the finished accumulator, 4 that warp has stored its part of the tile
// once: 8 kernel entered, 9 set-up done, 10 first operand load issued
#define TG_STAMP(tile, slot) do { if (pair == 0 && rank == 0 && (tile) < (unsigned)TG_TRACE_TILES) tg_trace[(tile) * 16 + (slot)] = clock64(); } while (0)
#else
#define TG_STAMP(tile, slot) do { } while (0)
#endif

namespace {

constexpr int TG_BM = 128, TG_BN = 256, TG_BK = 32;      // tile and samples per stage
constexpr int TG_STAGES = 4;
constexpr int TG_BOX_BYTES = 32 * TG_BK * 4;             // one 32-float x 32-row box: 4 KiB
constexpr int TG_A_BYTES = (TG_BM / 32) * TG_BOX_BYTES;  // 16 KiB
constexpr int TG_B_BYTES = (TG_BN / 32) * TG_BOX_BYTES;  // 32 KiB
constexpr int TG_STAGE_BYTES = TG_A_BYTES + TG_B_BYTES;  // 48 KiB
constexpr int TG_THREADS = 192;
constexpr int TG_TMEM_COLS = 512;                        // two accumulators of 256 fp32 columns
constexpr int TG_EPI_LD = 36;                            // padded row length of the epilogue staging (floats)
constexpr int TG_EPI_BYTES = 4 * 32 * TG_EPI_LD * 4;     // one 32 x 32 block per epilogue warp
constexpr size_t TG_SMEM_BYTES = (size_t)TG_STAGES * TG_STAGE_BYTES + TG_EPI_BYTES + 1024 /*alignment slack*/ + 256;

struct TgParams {
    int M, N, B;              // gw is M x N (M = neurons of the layer, N = neurons below = row length)
    int tiles_m, tiles_n;
    lf_sgd sgd;               // w_sub != nullptr: store w_sub - eta * (the contraction) instead
    float* gw;
    unsigned* status;
    unsigned long long budget_ns;
    int withhold;             // test hook (LF_OPT_WITHHOLD = 2): one producer leaves out the loads of its first
                              // stage, so that every wait behind it runs out
};

struct TgShared {
    unsigned long long full[TG_STAGES];
    unsigned long long empty[TG_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned tmem_base;
    volatile unsigned abort_flag;
};

// Bounded wait; returns false once this CTA has given up.
__device__ __forceinline__ bool tg_wait(unsigned bar, unsigned parity, const TgParams& P, TgShared* sh)
{
    if (lfptx::mbar_try_wait(bar, parity)) return true;
    if (sh->abort_flag) return false;
    const unsigned long long t0 = lfptx::globaltimer_ns();
    unsigned spins = 0;
    while (!lfptx::mbar_try_wait(bar, parity)) {
        if ((++spins & 15u) == 0u) {
            if (sh->abort_flag) return false;
            if (lfptx::globaltimer_ns() - t0 > P.budget_ns) {
                atomicOr(P.status, LF_DEV_TIMEOUT_BARRIER);
                sh->abort_flag = 1u;
                return false;
            }
        }
    }
    return true;
}
// Shared-memory matrix descriptor of an MN-major 32-bit operand (128-byte swizzle, 32-byte
// atoms): 32 floats (128 B) run along M/N, four consecutive samples form one 512-byte swizzle
// atom; the next 32 columns start `lbo` bytes further, the next four samples 512 bytes further.
__device__ __forceinline__ unsigned long long tg_make_desc(unsigned smem_addr, unsigned lbo_bytes)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);          // start address, bits [0,14)
    d |= (unsigned long long)((lbo_bytes >> 4) & 0x3FFFu) << 16;     // leading byte offset, bits [16,30)
    d |= (unsigned long long)((512u >> 4) & 0x3FFFu) << 32;          // stride byte offset, bits [32,46)
    d |= 1ull << 46;                                                 // descriptor version of this architecture
    d |= 1ull << 61;                                                 // layout type: 128-byte swizzle, 32-byte atoms
    return d;
}
// Instruction descriptor of kind::tf32: fp32 accumulator, TF32 x TF32, both operands MN-major.
__device__ __forceinline__ unsigned tg_make_idesc(int M, int Nn)
{
    unsigned d = 0;
    d |= 1u << 4;                       // accumulator format: F32
    d |= 2u << 7;                       // A format: TF32
    d |= 2u << 10;                      // B format: TF32
    d |= 1u << 15;                      // A is MN-major
    d |= 1u << 16;                      // B is MN-major
    d |= (unsigned)(Nn >> 3) << 17;     // N / 8
    d |= (unsigned)(M >> 4) << 24;      // M / 16
    return d;
}
__device__ __forceinline__ void tg_mma_tf32(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                            unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrive once all tensor-core operations issued so far by this thread have completed
__device__ __forceinline__ void tg_commit(unsigned bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}


// Fused weight update: ask L2 for the part of the w tile this warp will subtract from (32 rows x
// `cols` columns starting at row_first, col_first), one 128-byte line per request, while the
// tile is still being multiplied.
__device__ __forceinline__ void tg_prefetch_w(const float* w, int M, int N, int row_first, int col_first, int cols, int lane)
{
    const int row = row_first + lane;
    if (row >= M) return;
    const float* p = w + (size_t)row * N + col_first;
    for (int c = 0; c < cols && col_first + c < N; c += 32)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p + c));
}

__global__ void __launch_bounds__(TG_THREADS, 1)
k_gw_gemm_tf32(const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_a,
               const TgParams P)
{
    extern __shared__ unsigned char tg_smem_raw[];
    // operand stages must sit on 1024-byte boundaries (the swizzle atom)
    unsigned char* stages = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(tg_smem_raw) + 1023u) & ~(uintptr_t)1023u);
    float* epi = reinterpret_cast<float*>(stages + (size_t)TG_STAGES * TG_STAGE_BYTES);
    TgShared* sh = reinterpret_cast<TgShared*>(stages + (size_t)TG_STAGES * TG_STAGE_BYTES + TG_EPI_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = P.tiles_m * P.tiles_n;
    const int n_k = (P.B + TG_BK - 1) / TG_BK;

    if (threadIdx.x == 0) {
        for (int i = 0; i < TG_STAGES; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->tmem_full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->tmem_empty[i]), 128);
        }
        sh->abort_flag = 0u;
        lfptx::mbar_fence_init();
    }
    if (warp == 1) {   // tensor memory for both accumulators
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(lfptx::smem_u32(&sh->tmem_base)), "r"((unsigned)TG_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    lfptx::tc_fence_before();
    __syncthreads();
    lfptx::tc_fence_after();
    const unsigned tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------------------
        if (lane == 0) {
            unsigned it = 0;
            for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
                const int tm = t / P.tiles_n, tn = t - tm * P.tiles_n;
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    const unsigned st = it % TG_STAGES, use = it / TG_STAGES;
                    if (use > 0 && !tg_wait(lfptx::smem_u32(&sh->empty[st]), (use - 1) & 1u, P, sh)) break;
                    const unsigned bar = lfptx::smem_u32(&sh->full[st]);
                    lfptx::mbar_arrive_expect_tx(bar, TG_STAGE_BYTES);
                    if (P.withhold && blockIdx.x == 0 && it == 0) continue;   // test hook: armed, never loaded
                    const unsigned a_dst = lfptx::smem_u32(stages + (size_t)st * TG_STAGE_BYTES);
                    const unsigned b_dst = a_dst + TG_A_BYTES;
#pragma unroll
                    for (int i = 0; i < TG_BM / 32; ++i)
                        lfptx::tma_load_2d(a_dst + i * TG_BOX_BYTES, &map_d, bar, tm * TG_BM + i * 32, ks * TG_BK);
#pragma unroll
                    for (int i = 0; i < TG_BN / 32; ++i)
                        lfptx::tma_load_2d(b_dst + i * TG_BOX_BYTES, &map_a, bar, tn * TG_BN + i * 32, ks * TG_BK);
                }
                if (sh->abort_flag) break;
            }
            // after giving up: do not let the CTA exit under loads that are still landing
            if (sh->abort_flag) {
                const unsigned long long t0 = lfptx::globaltimer_ns();
                for (unsigned j = it > TG_STAGES ? it - TG_STAGES : 0; j < it; ++j) {
                    const unsigned bar = lfptx::smem_u32(&sh->full[j % TG_STAGES]);
                    while (!lfptx::mbar_try_wait(bar, (j / TG_STAGES) & 1u) && lfptx::globaltimer_ns() - t0 < 50000000ull) { }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer --------------------------------------------
        if (lane == 0) {
            const unsigned idesc = tg_make_idesc(TG_BM, TG_BN);
            unsigned it = 0, tile_i = 0;
            for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_i) {
                const unsigned ab = tile_i & 1u, ab_use = tile_i >> 1;
                if (ab_use > 0 && !tg_wait(lfptx::smem_u32(&sh->tmem_empty[ab]), (ab_use - 1) & 1u, P, sh)) break;
                lfptx::tc_fence_after();
                const unsigned d_tmem = tmem_base + ab * (unsigned)TG_BN;
                bool ok = true;
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    const unsigned st = it % TG_STAGES, use = it / TG_STAGES;
                    if (!tg_wait(lfptx::smem_u32(&sh->full[st]), use & 1u, P, sh)) { ok = false; break; }
                    lfptx::tc_fence_after();
                    const unsigned a_addr = lfptx::smem_u32(stages + (size_t)st * TG_STAGE_BYTES);
                    const unsigned b_addr = a_addr + TG_A_BYTES;
#pragma unroll
                    for (int kk = 0; kk < TG_BK / 8; ++kk) {      // eight samples per instruction
                        const unsigned long long da = tg_make_desc(a_addr + kk * 1024, TG_BOX_BYTES);
                        const unsigned long long db = tg_make_desc(b_addr + kk * 1024, TG_BOX_BYTES);
                        tg_mma_tf32(d_tmem, da, db, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                    }
                    tg_commit(lfptx::smem_u32(&sh->empty[st]));      // the stage may be refilled once these are done
                }
                if (!ok) break;
                tg_commit(lfptx::smem_u32(&sh->tmem_full[ab]));      // accumulator complete
            }
        }
    } else {
        // ------------------------------ epilogue (warps 2..5) ---------------------------------
        const int quad = warp & 3;                 // the TMEM lane quadrant this warp may read
        unsigned tile_i = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_i) {
            const int tm = t / P.tiles_n, tn = t - tm * P.tiles_n;
            const unsigned ab = tile_i & 1u, ab_use = tile_i >> 1;
            if (P.sgd.w_sub) tg_prefetch_w(P.sgd.w_sub, P.M, P.N, tm * TG_BM + quad * 32, tn * TG_BN, TG_BN, lane);
            if (!tg_wait(lfptx::smem_u32(&sh->tmem_full[ab]), ab_use & 1u, P, sh)) break;
            lfptx::tc_fence_after();
            // A thread reads one accumulator row (32 columns at a time).  The block is turned
            // through shared memory so that the warp stores whole 128-byte row segments.
            float* blk = epi + (warp - 2) * 32 * TG_EPI_LD;
            const int row0 = tm * TG_BM + quad * 32;
            const int sub_r = lane >> 3, sub_c = (lane & 7) * 4;
#pragma unroll 1
            for (int cchunk = 0; cchunk < TG_BN / 32; ++cchunk) {
                // fused weight update: the loads of w go out before the accumulator is fetched
                float4 wv[8];
                const int col_w = tn * TG_BN + cchunk * 32 + sub_c;
                if (P.sgd.w_sub && col_w < P.N) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (row0 + i * 4 + sub_r < P.M)
                            wv[i] = __ldcs(reinterpret_cast<const float4*>(P.sgd.w_sub + (size_t)(row0 + i * 4 + sub_r) * P.N + col_w));
                }
                unsigned r[32];
                lfptx::tmem_ld32(tmem_base + ((unsigned)(quad * 32) << 16) + ab * (unsigned)TG_BN + cchunk * 32, r);
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<float4*>(blk + lane * TG_EPI_LD + 4 * v) =
                        make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                    __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                __syncwarp();
                const int col = tn * TG_BN + cchunk * 32 + sub_c;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = i * 4 + sub_r;
                    float4 val = *reinterpret_cast<const float4*>(blk + rr * TG_EPI_LD + sub_c);
                    if (row0 + rr < P.M && col < P.N) {
                        const size_t off = (size_t)(row0 + rr) * P.N + col;
                        if (P.sgd.w_sub) val = lf_sgd_apply4(P.sgd.eta, wv[i], val);
                        __stcs(reinterpret_cast<float4*>(P.gw + off), val);
                    }
                }
                __syncwarp();
            }
            lfptx::tc_fence_before();
            lfptx::mbar_arrive(lfptx::smem_u32(&sh->tmem_empty[ab]));
        }
    }

    lfptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        lfptx::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((unsigned)TG_TMEM_COLS)
                     : "memory");
    }
}

// ================================================================================================
// Two-SM form for batches of at most 256 samples: a pair of CTAs (one thread-block cluster) works
// on 256 rows of gw at a time with tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 8; an
// instruction of this kind takes about as long for 128 columns as for 256, so tiles are 256 wide).
//   * The delta operand of the pair's 256 rows -- every sample of it, at most 128 KiB per CTA --
//     is loaded ONCE per row block and stays in shared memory while the pair walks along the
//     row block; only the activation operand streams (128 columns x 32 samples = 16 KiB per CTA
//     and stage), and the two CTAs read each other's half of it.  Per 128 KiB of gradient a CTA
//     stores it then loads 128 KiB of operands, against 384 KiB in the one-SM kernel above,
//     which waits for those loads (a multiprocessor takes in about 32 bytes per clock from L2).
//   * 256 x 256 pair tiles, each pair a contiguous run of them in row-major order; two
//     accumulators of 256 columns in tensor memory, so the epilogue of a tile overlaps the
//     next tile's multiplications.
// Hand-offs between the two CTAs: both producers credit their loads to the LEADER's (rank 0)
// "full" barriers; the leader's tcgen05.commit reaches the "empty" / "accumulator full" barriers
// of both CTAs at once; the epilogue warps of both CTAs arrive on the leader's "accumulator
// empty" barrier.  All waits are bounded as above.
constexpr int TP_BM = 128;                               // rows of gw per CTA (256 per pair)
constexpr int TP_BN = 256;                               // columns of a pair tile (128 loaded per CTA)
constexpr int TP_MAX_KS = 8;                             // at most 8 x 32 = 256 samples
constexpr int TP_STAGES = 3;
constexpr int TPS_STAGES = 5;                             // streaming form (B > 256): stages of 32 KiB, both operands
constexpr int TP_ACC = 2;                                // accumulators of TP_BN columns
constexpr int TP_A_STAGE_BYTES = (TP_BM / 32) * TG_BOX_BYTES;        // 16 KiB: 128 rows x 32 samples
constexpr int TP_B_STAGE_BYTES = (TP_BN / 2 / 32) * TG_BOX_BYTES;    // 16 KiB: 128 columns x 32 samples
constexpr int TP_A_BYTES = TP_MAX_KS * TP_A_STAGE_BYTES;             // 128 KiB
constexpr int TP_THREADS = 320;                          // producer, issuer, eight epilogue warps
constexpr int TP_EPI_BYTES = 8 * 32 * TG_EPI_LD * 4;    // one 32 x 32 block per epilogue warp
constexpr size_t TP_SMEM_BYTES = (size_t)TP_A_BYTES + (size_t)TP_STAGES * TP_B_STAGE_BYTES + TP_EPI_BYTES +
                                 1024 /*alignment slack*/ + 512;
static_assert((size_t)TPS_STAGES * (TP_A_STAGE_BYTES + TP_B_STAGE_BYTES) <= (size_t)TP_A_BYTES + (size_t)TP_STAGES * TP_B_STAGE_BYTES,
              "the streaming form's ring overlays the resident operand and the activation ring");

struct TpShared {
    unsigned long long a_full[TP_MAX_KS];   // leader: delta operand chunk ks of both CTAs has landed
    unsigned long long a_empty;             // both: the resident delta operand may be replaced
    unsigned long long b_full[TPS_STAGES];  // leader: stage of both CTAs has landed
    unsigned long long b_empty[TPS_STAGES]; // both: stage may be refilled
    unsigned long long acc_full[TP_ACC];    // both: accumulator complete
    unsigned long long acc_empty[TP_ACC];   // leader: accumulator drained by both CTAs
    unsigned tmem_base;
    volatile unsigned abort_flag;
    // what this CTA's producer has issued (read by the leader when a launch is given up)
    unsigned prog_it;         // stage loads issued
    unsigned prog_a_loads;    // resident form: loads of the delta operand begun ...
    unsigned prog_a_ks;       // ... and chunks of the last one issued
};
static_assert(sizeof(TpShared) <= 512, "the barrier block must fit into the space reserved for it");

__device__ __forceinline__ void tp_mma_tf32(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                            unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair once every
// tensor-core operation issued so far has completed
__device__ __forceinline__ void tp_commit_both(unsigned bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void tp_arrive_remote(unsigned cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tp_complete_tx(unsigned bar, unsigned bytes)   // bytes that will never arrive
{
    asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ unsigned tp_ld_remote(unsigned cluster_addr)
{
    unsigned v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
    return v;
}
// Bounded wait on a barrier of this CTA; returns false once this CTA has given up.
__device__ __forceinline__ bool tp_wait(unsigned bar, unsigned parity, const TgParams& P, TpShared* sh)
{
    if (lfptx::mbar_try_wait_cluster(bar, parity)) return true;
    if (sh->abort_flag) return false;
    const unsigned long long t0 = lfptx::globaltimer_ns();
    unsigned spins = 0;
    while (!lfptx::mbar_try_wait_cluster(bar, parity)) {
        if ((++spins & 15u) == 0u) {
            if (sh->abort_flag) return false;
            if (lfptx::globaltimer_ns() - t0 > P.budget_ns || (((spins & 1023u) == 0u) && *((volatile unsigned*)P.status) != 0u)) {
                atomicOr(P.status, LF_DEV_TIMEOUT_BARRIER);
                sh->abort_flag = 1u;
                return false;
            }
        }
    }
    return true;
}

// RESIDENT = true: B <= 256, the delta operand of a row block stays in shared memory (above).
// RESIDENT = false: any B.  Both operands stream: a stage holds 32 samples of the pair's 256 rows of
// delta and 256 columns of a, half of each loaded by either CTA (32 KiB per CTA and stage, five
// stages over the same shared memory).  Per multiply-add a CTA then loads two thirds of what the
// one-SM kernel loads, which is what that kernel waits for at large B.
template <bool RESIDENT>
__global__ void __launch_bounds__(TP_THREADS, 1)
k_gw_gemm_tf32_pair(const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_a,
                    const TgParams P)
{
    extern __shared__ unsigned char tg_smem_raw[];
    // Both CTAs of the pair must use the same offsets (the tensor core applies one descriptor to
    // both); the dynamic shared memory starts at the same address in every CTA of a launch.
    unsigned char* a_res = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(tg_smem_raw) + 1023u) & ~(uintptr_t)1023u);
    unsigned char* b_ring = a_res + TP_A_BYTES;
    float* epi = reinterpret_cast<float*>(b_ring + (size_t)TP_STAGES * TP_B_STAGE_BYTES);
    TpShared* sh = reinterpret_cast<TpShared*>(reinterpret_cast<unsigned char*>(epi) + TP_EPI_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned rank = lfptx::cluster_ctarank();          // 0 = leader (issues the multiplications)
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int n_k = (P.B + TG_BK - 1) / TG_BK;        // RESIDENT: <= TP_MAX_KS
    constexpr unsigned N_ST = RESIDENT ? TP_STAGES : TPS_STAGES;
    const int n_tiles = P.tiles_m * P.tiles_n;        // tiles_m counts 256-row blocks here
    const int t_begin = (int)(((long long)n_tiles * pair) / n_pairs);
    const int t_end = (int)(((long long)n_tiles * (pair + 1)) / n_pairs);
    if (threadIdx.x == 0) TG_STAMP(0u, 8);

    if (threadIdx.x == 0) {
        for (int i = 0; i < TP_MAX_KS; ++i) lfptx::mbar_init(lfptx::smem_u32(&sh->a_full[i]), 1);
        lfptx::mbar_init(lfptx::smem_u32(&sh->a_empty), 1);
        for (int i = 0; i < TPS_STAGES; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->b_full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->b_empty[i]), 1);
        }
        for (int i = 0; i < TP_ACC; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->acc_full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->acc_empty[i]), 16);  // eight epilogue warps of each CTA
        }
        sh->abort_flag = 0u;
        lfptx::mbar_fence_init();
    }
    if (warp == 1) {   // tensor memory for the accumulators, the same columns in both CTAs
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(lfptx::smem_u32(&sh->tmem_base)), "r"((unsigned)(TP_ACC * TP_BN)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    lfptx::tc_fence_before();
    __syncthreads();
    lfptx::cluster_sync_all();   // the peer's barriers exist before anything can arrive on them
    lfptx::tc_fence_after();
    const unsigned tmem_base = sh->tmem_base;
    if (threadIdx.x == 0) TG_STAMP(0u, 9);

    if (warp == 0) {
        // ------------------------------ TMA producer (each CTA, its own halves) ----------------
        if (lane == 0) {
            unsigned it = 0, a_loads = 0, a_ks = 0;
            int cur_rb = -1;
            TG_STAMP(0u, 10);
            const int my_row0 = (int)rank * TP_BM;
            const int my_col0 = (int)rank * (TP_BN / 2);
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int rb = t / P.tiles_n, tn = t - rb * P.tiles_n;
                const bool new_rb = RESIDENT && rb != cur_rb;
                if (new_rb) {
                    // the resident delta operand changes: wait until every multiplication that
                    // reads the old one is done
                    if (a_loads > 0 && !tp_wait(lfptx::smem_u32(&sh->a_empty), (a_loads - 1) & 1u, P, sh)) break;
                    cur_rb = rb;
                    ++a_loads;
                    a_ks = 0;
                }
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    if (new_rb) {
                        ++a_ks;
                        const unsigned lbar = lfptx::smem_u32(&sh->a_full[ks]);
                        if (rank == 0) lfptx::mbar_arrive_expect_tx(lbar, 2u * TP_A_STAGE_BYTES);
                        const unsigned bar = lfptx::map_to_cta(lbar, 0);
                        const unsigned dst = lfptx::smem_u32(a_res + (size_t)ks * TP_A_STAGE_BYTES);
#pragma unroll
                        for (int i = 0; i < TP_BM / 32; ++i)
                            lfptx::tma_load_2d_pair(dst + i * TG_BOX_BYTES, &map_d, bar, rb * 2 * TP_BM + my_row0 + i * 32,
                                           ks * TG_BK);
                    }
                    const unsigned st = it % N_ST, use = it / N_ST;
                    if (use > 0 && !tp_wait(lfptx::smem_u32(&sh->b_empty[st]), (use - 1) & 1u, P, sh)) { ok = false; break; }
                    const unsigned lbar = lfptx::smem_u32(&sh->b_full[st]);
                    const unsigned bar = lfptx::map_to_cta(lbar, 0);
                    if (P.withhold && pair == 0 && rank == 1 && it == 0) continue;   // test hook: the peer leaves out its first stage
                    if (RESIDENT) {
                        if (rank == 0) lfptx::mbar_arrive_expect_tx(lbar, 2u * TP_B_STAGE_BYTES);
                        const unsigned dst = lfptx::smem_u32(b_ring + (size_t)st * TP_B_STAGE_BYTES);
#pragma unroll
                        for (int i = 0; i < TP_BN / 2 / 32; ++i)
                            lfptx::tma_load_2d_pair(dst + i * TG_BOX_BYTES, &map_a, bar, tn * TP_BN + my_col0 + i * 32, ks * TG_BK);
                    } else {
                        // streaming form: this CTA's half of both operands for these 32 samples
                        if (rank == 0) lfptx::mbar_arrive_expect_tx(lbar, 2u * (TP_A_STAGE_BYTES + TP_B_STAGE_BYTES));
                        const unsigned dst_a = lfptx::smem_u32(a_res + (size_t)st * (TP_A_STAGE_BYTES + TP_B_STAGE_BYTES));
                        const unsigned dst_b = dst_a + TP_A_STAGE_BYTES;
#pragma unroll
                        for (int i = 0; i < TP_BM / 32; ++i)
                            lfptx::tma_load_2d_pair(dst_a + i * TG_BOX_BYTES, &map_d, bar, rb * 2 * TP_BM + my_row0 + i * 32,
                                           ks * TG_BK);
#pragma unroll
                        for (int i = 0; i < TP_BN / 2 / 32; ++i)
                            lfptx::tma_load_2d_pair(dst_b + i * TG_BOX_BYTES, &map_a, bar, tn * TP_BN + my_col0 + i * 32, ks * TG_BK);
                    }
                }
            }
            sh->prog_it = it; sh->prog_a_loads = a_loads; sh->prog_a_ks = a_ks;
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (leader CTA only) ---------------------------
        if (lane == 0 && rank == 0) {
            const unsigned idesc = tg_make_idesc(2 * TP_BM, TP_BN);
            unsigned it = 0, tile_i = 0, a_loads = 0;
            int cur_rb = -1;
            for (int t = t_begin; t < t_end; ++t, ++tile_i) {
                const int rb = t / P.tiles_n;
                const bool new_rb = RESIDENT && rb != cur_rb;
                if (new_rb) { cur_rb = rb; ++a_loads; }
                const unsigned ab = tile_i % TP_ACC, ab_use = tile_i / TP_ACC;
                if (ab_use > 0 && !tp_wait(lfptx::smem_u32(&sh->acc_empty[ab]), (ab_use - 1) & 1u, P, sh)) break;
                lfptx::tc_fence_after();
                TG_STAMP(tile_i, 0);
                const unsigned d_tmem = tmem_base + ab * (unsigned)TP_BN;
                bool ok = true;
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    if (new_rb && !tp_wait(lfptx::smem_u32(&sh->a_full[ks]), (a_loads - 1) & 1u, P, sh)) { ok = false; break; }
                    const unsigned st = it % N_ST, use = it / N_ST;
                    if (!tp_wait(lfptx::smem_u32(&sh->b_full[st]), use & 1u, P, sh)) { ok = false; break; }
                    if (ks == 0) TG_STAMP(tile_i, 1);
                    lfptx::tc_fence_after();
                    const unsigned a_addr = RESIDENT ? lfptx::smem_u32(a_res + (size_t)ks * TP_A_STAGE_BYTES)
                                                     : lfptx::smem_u32(a_res + (size_t)st * (TP_A_STAGE_BYTES + TP_B_STAGE_BYTES));
                    const unsigned b_addr = RESIDENT ? lfptx::smem_u32(b_ring + (size_t)st * TP_B_STAGE_BYTES)
                                                     : a_addr + TP_A_STAGE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < TG_BK / 8; ++kk) {      // eight samples per instruction
                        const unsigned long long da = tg_make_desc(a_addr + kk * 1024, TG_BOX_BYTES);
                        const unsigned long long db = tg_make_desc(b_addr + kk * 1024, TG_BOX_BYTES);
                        tp_mma_tf32(d_tmem, da, db, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                    }
                    tp_commit_both(lfptx::smem_u32(&sh->b_empty[st]));
                }
                if (!ok) break;
                // the last tile of a row block frees the resident operand for the next one
                if (RESIDENT && t + 1 < t_end && (t + 1) / P.tiles_n != rb) tp_commit_both(lfptx::smem_u32(&sh->a_empty));
                tp_commit_both(lfptx::smem_u32(&sh->acc_full[ab]));
                TG_STAMP(tile_i, 2);
            }
        }
    } else {
        // ------------------------------ epilogue (warps 2..9 of both CTAs) ---------------------
        // Two warps per TMEM lane quadrant, each taking 128 of the tile's 256 columns in blocks
        // of 32 x 32 that are turned through shared memory, so that a warp stores whole 128-byte
        // row segments.
        const int quad = warp & 3;                 // the TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;
        const unsigned leader_acc_empty0 = lfptx::map_to_cta(lfptx::smem_u32(&sh->acc_empty[0]), 0);
        float* blk = epi + (warp - 2) * 32 * TG_EPI_LD;
        const int sub_r = lane >> 3, sub_c = (lane & 7) * 4;
        unsigned tile_i = 0;
        for (int t = t_begin; t < t_end; ++t, ++tile_i) {
            const int rb = t / P.tiles_n, tn = t - rb * P.tiles_n;
            const unsigned ab = tile_i % TP_ACC, ab_use = tile_i / TP_ACC;
            const int row0 = rb * 2 * TP_BM + (int)rank * TP_BM + quad * 32 + sub_r;
            const int col0 = tn * TP_BN + half * (TP_BN / 2) + sub_c;
            const size_t out_off = (size_t)row0 * P.N + col0;
            float* out_row = P.gw + out_off;
            const float* w_row = P.sgd.w_sub ? P.sgd.w_sub + out_off : nullptr;
            const size_t row_step = (size_t)4 * P.N;
            if (w_row)
                tg_prefetch_w(P.sgd.w_sub, P.M, P.N, row0 - sub_r, tn * TP_BN + half * (TP_BN / 2), TP_BN / 2, lane);
            if (!tp_wait(lfptx::smem_u32(&sh->acc_full[ab]), ab_use & 1u, P, sh)) break;
            if (threadIdx.x == 64) TG_STAMP(tile_i, 3);
            lfptx::tc_fence_after();
#pragma unroll 1
            for (int cchunk = 0; cchunk < TP_BN / 2 / 32; ++cchunk) {
                // fused weight update: the loads of w go out before the accumulator is fetched
                float4 wv[8];
                if (w_row && col0 + cchunk * 32 < P.N) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (row0 + i * 4 < P.M)
                            wv[i] = __ldcs(reinterpret_cast<const float4*>(w_row + i * row_step + cchunk * 32));
                }
                unsigned r[32];
                lfptx::tmem_ld32(tmem_base + ((unsigned)(quad * 32) << 16) + ab * (unsigned)TP_BN + half * (TP_BN / 2) + cchunk * 32, r);
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<float4*>(blk + lane * TG_EPI_LD + 4 * v) =
                        make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                    __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                __syncwarp();
                if (col0 + cchunk * 32 < P.N) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float4 val = *reinterpret_cast<const float4*>(blk + (i * 4 + sub_r) * TG_EPI_LD + sub_c);
                        if (row0 + i * 4 < P.M) {
                            if (w_row) val = lf_sgd_apply4(P.sgd.eta, wv[i], val);
                            __stcs(reinterpret_cast<float4*>(out_row + i * row_step + cchunk * 32), val);
                        }
                    }
                }
                __syncwarp();
            }
            lfptx::tc_fence_before();
            __syncwarp();
            if (threadIdx.x == 64) TG_STAMP(tile_i, 4);
            if (lane == 0) tp_arrive_remote(leader_acc_empty0 + ab * (unsigned)sizeof(unsigned long long));
        }
    }

    // Neither CTA may leave (or free tensor memory) while the other can still reach it: the
    // leader's multiplications read the peer's shared memory and write the peer's tensor
    // memory, and its commits arrive on the peer's barriers.
    lfptx::tc_fence_before();
    __syncthreads();
    lfptx::cluster_sync_all();     // both producers have stopped; what each has issued is in its prog_* words
    if (threadIdx.x == 0 && rank == 0) {
        // A launch that was given up: no CTA of the pair may exit while operand loads are still on
        // their way into its shared memory.  The loads of BOTH CTAs are credited to the leader's
        // barriers, so the leader can see all of them land -- once every phase that anyone issued
        // loads for has been brought to a state it can complete in: a phase only the peer loaded
        // for gets the arrival (and the byte count) the leader never gave it, a phase only the
        // leader loaded for is told that the peer's bytes will not come.  Then wait, with a limit.
        const bool gave_up = sh->abort_flag != 0u || tp_ld_remote(lfptx::map_to_cta(lfptx::smem_u32((const void*)&sh->abort_flag), 1)) != 0u;
        if (gave_up) {
            const unsigned it_l = sh->prog_it, it_p = tp_ld_remote(lfptx::map_to_cta(lfptx::smem_u32(&sh->prog_it), 1));
            const unsigned stage_bytes = RESIDENT ? (unsigned)TP_B_STAGE_BYTES : (unsigned)(TP_A_STAGE_BYTES + TP_B_STAGE_BYTES);
            const unsigned it_hi = it_l > it_p ? it_l : it_p, it_lo = it_l < it_p ? it_l : it_p;
            for (unsigned j = it_lo; j < it_hi; ++j) {
                const unsigned bar = lfptx::smem_u32(&sh->b_full[j % N_ST]);
                if (j >= it_l) lfptx::mbar_arrive_expect_tx(bar, stage_bytes);      // only the peer loaded
                else tp_complete_tx(bar, stage_bytes);                  // only the leader loaded
            }
            const unsigned long long t0 = lfptx::globaltimer_ns();
            for (unsigned j = it_hi > N_ST ? it_hi - N_ST : 0; j < it_hi; ++j) {
                const unsigned bar = lfptx::smem_u32(&sh->b_full[j % N_ST]);
                while (!lfptx::mbar_try_wait(bar, (j / N_ST) & 1u) && lfptx::globaltimer_ns() - t0 < 50000000ull) { }
            }
            if (RESIDENT) {
                // the resident operand: chunks of the load that was under way (loads before it were
                // waited for by the multiplications that freed the operand for this one)
                const unsigned al_l = sh->prog_a_loads, al_p = tp_ld_remote(lfptx::map_to_cta(lfptx::smem_u32(&sh->prog_a_loads), 1));
                const unsigned ak_l = sh->prog_a_ks, ak_p = tp_ld_remote(lfptx::map_to_cta(lfptx::smem_u32(&sh->prog_a_ks), 1));
                const unsigned al = al_l > al_p ? al_l : al_p;
                const unsigned kl = al_l == al ? ak_l : 0u, kp = al_p == al ? ak_p : 0u;   // chunks of load `al`
                for (unsigned ks = 0; ks < (kl > kp ? kl : kp) && al > 0; ++ks) {
                    const unsigned bar = lfptx::smem_u32(&sh->a_full[ks]);
                    if (ks >= kl) lfptx::mbar_arrive_expect_tx(bar, (unsigned)TP_A_STAGE_BYTES);
                    else if (ks >= kp) tp_complete_tx(bar, (unsigned)TP_A_STAGE_BYTES);
                    while (!lfptx::mbar_try_wait(bar, (al - 1) & 1u) && lfptx::globaltimer_ns() - t0 < 50000000ull) { }
                }
            }
        }
    }
    lfptx::cluster_sync_all();
    if (warp == 1) {
        lfptx::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((unsigned)(TP_ACC * TP_BN)) : "memory");
    }
}


typedef CUresult (*tg_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

tg_encode_fn tg_get_encode()
{
    static tg_encode_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<tg_encode_fn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// [B][N] fp32 matrix as a 2-D tensor map with 32-float x 32-row boxes, 128-byte swizzle of 32-byte atoms.
bool tg_encode_operand(CUtensorMap* m, const float* base, int N, int B)
{
    cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)B};
    cuuint64_t strides[1] = {(cuuint64_t)N * 4};
    cuuint32_t box[2] = {32, (cuuint32_t)TG_BK};
    cuuint32_t estr[2] = {1, 1};
    return tg_get_encode()(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Largest number of CTA pairs of the two-SM kernel that can be resident at once (0: unusable).
// Queried once per device; also opts the kernel in to its dynamic shared memory.
static int tp_max_pairs(const lf_ctx* c)
{
    static int cached_dev = -1, cached = 0;
    if (cached_dev == c->device) return cached;
    int n = 0;
    if ((size_t)c->smem_optin >= TP_SMEM_BYTES &&
        cudaFuncSetAttribute(k_gw_gemm_tf32_pair<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)TP_SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(k_gw_gemm_tf32_pair<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)TP_SMEM_BYTES) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        cfg.gridDim = dim3(2 * 16); cfg.blockDim = dim3(TP_THREADS); cfg.dynamicSmemBytes = TP_SMEM_BYTES;
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n_stream = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_gw_gemm_tf32_pair<true>, &cfg) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n_stream, k_gw_gemm_tf32_pair<false>, &cfg) != cudaSuccess)
            n = 0;
        else if (n_stream < n)
            n = n_stream;
    }
    cudaGetLastError();
    cached_dev = c->device; cached = n;
    return n;
}

bool lf_tf32_supported(const lf_ctx* c)
{
    if (c->B < 2) return false;
    if ((size_t)c->smem_optin < TG_SMEM_BYTES) return false;
    if (!tg_get_encode()) return false;
    // opt in to the large dynamic shared memory once per device (not during a stream capture)
    static int attr_dev = -1;
    if (attr_dev != c->device) {
        if (cudaFuncSetAttribute(k_gw_gemm_tf32, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)TG_SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        attr_dev = c->device;
    }
    tp_max_pairs(c);
    return true;
}

int lf_gw_gemm_tf32(lf_ctx* c, const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                    lf_sgd sgd, cudaStream_t s, int* launches)
{
    // delta_l is [B][n_out], a_prev is [B][n_in], gw_l is n_out x n_in
    alignas(64) CUtensorMap map_d, map_a;
    if (!tg_encode_operand(&map_d, delta_l, n_out, c->B) || !tg_encode_operand(&map_a, a_prev, n_in, c->B)) {
        c->last_cuda_error = (int)cudaErrorInvalidValue;
        return LF_ECUDA;
    }
    TgParams P;
    P.M = n_out; P.N = n_in; P.B = c->B;
    P.gw = gw_l;
    P.sgd = sgd;
    P.status = c->status_dev;
    P.budget_ns = (unsigned long long)c->wait_budget_us * 1000ull;
    P.withhold = c->withhold == 2 ? 1 : 0;
    const int max_pairs = c->tc_pair_kernels ? tp_max_pairs(c) : 0;
    if (max_pairs > 0) {
        // two-SM kernels: up to 256 samples the delta operand of a 256-row block stays in shared
        // memory; beyond, both operands stream
        P.tiles_m = (n_out + 2 * TP_BM - 1) / (2 * TP_BM);
        P.tiles_n = (n_in + TP_BN - 1) / TP_BN;
        const int tiles = P.tiles_m * P.tiles_n;
        const int pairs = tiles < max_pairs ? tiles : max_pairs;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(TP_THREADS); cfg.dynamicSmemBytes = TP_SMEM_BYTES;
        cfg.stream = s;
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        if (c->B <= TP_MAX_KS * TG_BK)
            LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_gw_gemm_tf32_pair<true>, map_d, map_a, P));
        else
            LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_gw_gemm_tf32_pair<false>, map_d, map_a, P));
        c->stats.gw_tiling = LF_TC_TILING_TWO_SM;
        *launches += 1;
        return LF_OK;
    }
    P.tiles_m = (n_out + TG_BM - 1) / TG_BM;
    P.tiles_n = (n_in + TG_BN - 1) / TG_BN;
    const int tiles = P.tiles_m * P.tiles_n;
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    k_gw_gemm_tf32<<<grid, TG_THREADS, TG_SMEM_BYTES, s>>>(map_d, map_a, P);
    LF_CUDA_TRY(c, cudaGetLastError());
    c->stats.gw_tiling = LF_TC_TILING_ONE_SM;
    *launches += 1;
    return LF_OK;
}

void lf_tf32_release(lf_ctx*) {}
