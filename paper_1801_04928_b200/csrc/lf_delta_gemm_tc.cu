// Mini-batch delta recurrence (Eq. bp2 for B > 1) on the tensor cores at fp32 accuracy:
//     T[b][n] = sum_j D[b][j] * W[j][n],   delta^l[b][n] = T[b][n] * a^l[b][n] (1 - a^l[b][n])
// with D = delta^{l+1} [B][N] and W = w^{l+1} [N][N] (row j, column n).  The same kernel, with
// the W operand read K-major instead, does the mini-batch forward contraction (Eq. z):
//     Z[b][n] = sum_j A[b][j] * W[n][j] + bias[n],   A = a^{l-1}, W = w^l.
//
// A TF32 product keeps 11 significant bits, far too few for the 1e-5 gate on delta, so every
// operand x is split in shared memory into hi = tf32(x) (round to nearest) and lo = x - hi
// (exact in fp32) and three products are accumulated in fp32: lo*hi + hi*lo + hi*hi; the
// dropped lo*lo term and the truncation of lo are of relative size 2^-22.  The tensor core
// adds into its fp32 accumulator by truncation, which biases long accumulations (about 1e-5
// relative after 768 instructions); therefore an accumulator in tensor memory only ever holds
// the 12 instructions of one 32-wide K stage (small terms first), and the stage results are
// added in registers with round-to-nearest (two accumulators in TMEM, used alternately, so
// the adding overlaps the next stage's instructions).
//
// Work unit = (128 samples) x (128 columns n) x (one K split of the j range); one CTA per unit,
// units dealt round-robin.  Warp 0: TMA producer (D as K-major 128-byte-swizzled rows, W as
// MN-major boxes in the 128-byte swizzle with 32-byte atoms).  Warps 2-5: split each stage in
// place (hi overwrites the raw tile, lo goes beside it), then act as the epilogue.  Warp 1:
// issues the tcgen05.mma kind::tf32 instructions (M = 128, N = 128, K = 8), accumulator in TMEM.
// Partial results of the K splits go to scratch; k_delta_finish adds them in split order and
// applies sigma'.  All waits are bounded; on expiry the status word is raised.
#include <cuda.h>

#include "lf_internal.h"
#include "lf_ptx.cuh"

// Debug builds (-DLF_DG_TRACE): the leader CTA of pair 0 of the two-SM kernel stamps its SM clock at
// nine points of each of its first DG_TRACE_STAGES K stages (see DG_STAMP below); the release
// library carries none of this.
#ifdef LF_DG_TRACE
constexpr int DG_TRACE_STAGES = 128;
__device__ long long dg_trace[DG_TRACE_STAGES * 16];
extern "C" int lf_debug_read_pair_trace(long long* out)
{
    if (!out) return LF_ENULL;
    cudaDeviceSynchronize();
    return cudaMemcpyFromSymbol(out, dg_trace, sizeof(dg_trace)) == cudaSuccess ? LF_OK : LF_ECUDA;
}
// 0 loads issued, 1 loads landed, 2 second-ring slot free, 3 split written, 4 issuer sees the split,
// 5 issuer has the accumulator, 6 products and commits issued, 7 products done, 8 accumulator drained
#define DG_STAMP(slot) do { if (pair == 0 && rank == 0 && it < (unsigned)DG_TRACE_STAGES) dg_trace[it * 16 + (slot)] = clock64(); } while (0)
// once per launch, in the words 9 .. 12 of stage 0: 9 kernel entered, 10 set-up done (barriers, tensor
// memory, cluster barrier), 11 a summing warp has written its last partial sums, 12 before the exit
#define DG_STAMP_ONCE(slot) do { if (pair == 0 && rank == 0 && (threadIdx.x == 256 || ((slot) < 11 && threadIdx.x == 0))) dg_trace[slot] = clock64(); } while (0)
#else
#define DG_STAMP(slot) do { } while (0)
#define DG_STAMP_ONCE(slot) do { } while (0)
#endif

namespace {

constexpr int DG_BM = 128, DG_BN = 128, DG_BK = 32;
constexpr int DG_STAGES = 3;
constexpr int DG_A_BYTES = DG_BM * DG_BK * 4;            // 16 KiB: 128 rows of 128 bytes
constexpr int DG_BOX_BYTES = 32 * DG_BK * 4;             // 4 KiB: 32 columns x 32 rows of W
constexpr int DG_B_BYTES = (DG_BN / 32) * DG_BOX_BYTES;  // 16 KiB
constexpr int DG_RAW_BYTES = DG_A_BYTES + DG_B_BYTES;    // what TMA delivers per stage
constexpr int DG_STAGE_BYTES = 2 * DG_RAW_BYTES;         // hi (in place) + lo
constexpr int DG_THREADS = 192;
constexpr int DG_TMEM_COLS = 256;                        // two stage accumulators of 128 columns
constexpr int DG_EPI_LD = 36;
constexpr int DG_EPI_BYTES = 4 * 32 * DG_EPI_LD * 4;
constexpr size_t DG_SMEM_BYTES = (size_t)DG_STAGES * DG_STAGE_BYTES + DG_EPI_BYTES + 1024 + 256;

struct DgParams {
    int N, B;                 // the output is [B][N]; the contraction length reaches the kernels only
                              // through the K-block counts below (loads beyond it are zero-filled)
    int tiles_m, tiles_n, splits;
    int k_per_split;          // j range of one split (multiple of DG_BK)
    int kb_per_tile;          // two-SM kernel: K blocks (of DG_BK) of one tile
    int g_total;              // two-SM kernel: tiles * kb_per_tile, dealt to the pairs in contiguous runs
    float* partial;           // [splits][B][N]
    unsigned* status;
    unsigned long long budget_ns;
};

struct DgShared {
    unsigned long long full[DG_STAGES];    // TMA landed
    unsigned long long split_done[DG_STAGES];  // hi/lo written (128 arrivals)
    unsigned long long empty[DG_STAGES];   // MMAs that read the stage are done
    unsigned long long acc_full[2], acc_empty[2];   // stage accumulator p holds a finished stage / is drained
    unsigned tmem_base;
    volatile unsigned abort_flag;
};

__device__ __forceinline__ bool dg_wait(unsigned bar, unsigned parity, const DgParams& P, DgShared* sh)
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
// K-major operand, 128-byte swizzle: rows of 128 bytes (32 floats along K), eight rows per
// 1024-byte atom (SBO); one instruction consumes 32 bytes of every row.
__device__ __forceinline__ unsigned long long dg_desc_kmajor(unsigned smem_addr)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);
    d |= (unsigned long long)1 << 16;                                // LBO: not used by swizzled K-major
    d |= (unsigned long long)((1024u >> 4) & 0x3FFFu) << 32;         // SBO: next group of eight rows
    d |= 1ull << 46;
    d |= 2ull << 61;                                                 // 128-byte swizzle
    return d;
}
// MN-major 32-bit operand, 128-byte swizzle with 32-byte atoms: 32 floats along N per row,
// four K rows per 512-byte atom (SBO), next 32 columns 4 KiB further (LBO).
__device__ __forceinline__ unsigned long long dg_desc_mnmajor(unsigned smem_addr)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);
    d |= (unsigned long long)((DG_BOX_BYTES >> 4) & 0x3FFFu) << 16;
    d |= (unsigned long long)((512u >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= 1ull << 61;
    return d;
}
// descriptor of the W tile for K step kk (eight values of the contraction index)
template <bool W_KMAJOR>
__device__ __forceinline__ unsigned long long dg_desc_w(unsigned tile_addr, int kk)
{
    return W_KMAJOR ? dg_desc_kmajor(tile_addr + kk * 32) : dg_desc_mnmajor(tile_addr + kk * 1024);
}
__device__ __forceinline__ unsigned dg_idesc(bool w_kmajor)
{
    unsigned d = 0;
    d |= 1u << 4;                             // fp32 accumulator
    d |= 2u << 7;                             // A: TF32
    d |= 2u << 10;                            // B: TF32
    d |= 0u << 15;                            // A is K-major
    d |= (w_kmajor ? 0u : 1u) << 16;          // B operand: K-major or MN-major
    d |= (unsigned)(DG_BN >> 3) << 17;
    d |= (unsigned)(DG_BM >> 4) << 24;
    return d;
}
__device__ __forceinline__ void dg_mma(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                       unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void dg_commit(unsigned bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ float dg_tf32_rn(float x)
{
    unsigned r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// W_KMAJOR = false: T = D * W   (Eq. bp2: w^{l+1}[j][n], contraction over its rows j; MN-major operand)
// W_KMAJOR = true : T = D * W^T (Eq. z:  w^l[n][j],     contraction over its columns j; K-major operand)
template <bool W_KMAJOR>
__global__ void __launch_bounds__(DG_THREADS, 1)
k_delta_gemm_tc(const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_w,
                const DgParams P)
{
    extern __shared__ unsigned char dg_smem_raw[];
    unsigned char* stages = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(dg_smem_raw) + 1023u) & ~(uintptr_t)1023u);
    float* epi = reinterpret_cast<float*>(stages + (size_t)DG_STAGES * DG_STAGE_BYTES);
    DgShared* sh = reinterpret_cast<DgShared*>(stages + (size_t)DG_STAGES * DG_STAGE_BYTES + DG_EPI_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_units = P.tiles_m * P.tiles_n * P.splits;
    const int n_k = P.k_per_split / DG_BK;

    if (threadIdx.x == 0) {
        for (int i = 0; i < DG_STAGES; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->split_done[i]), 128);
            lfptx::mbar_init(lfptx::smem_u32(&sh->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->acc_full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->acc_empty[i]), 128);
        }
        sh->abort_flag = 0u;
        lfptx::mbar_fence_init();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(lfptx::smem_u32(&sh->tmem_base)), "r"((unsigned)DG_TMEM_COLS) : "memory");
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
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                const int tn = u % P.tiles_n, tm = (u / P.tiles_n) % P.tiles_m, sp = u / (P.tiles_n * P.tiles_m);
                const int j0 = sp * P.k_per_split;
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    const unsigned st = it % DG_STAGES, use = it / DG_STAGES;
                    if (use > 0 && !dg_wait(lfptx::smem_u32(&sh->empty[st]), (use - 1) & 1u, P, sh)) break;
                    const unsigned bar = lfptx::smem_u32(&sh->full[st]);
                    lfptx::mbar_arrive_expect_tx(bar, DG_RAW_BYTES);
                    const unsigned a_dst = lfptx::smem_u32(stages + (size_t)st * DG_STAGE_BYTES);
                    // boxes of 32 rows: the loads of one box are few at a time, several boxes go side by side
#pragma unroll
                    for (int i = 0; i < DG_BM / 32; ++i)
                        lfptx::tma_load_2d(a_dst + i * DG_BOX_BYTES, &map_d, bar, j0 + ks * DG_BK, tm * DG_BM + i * 32);
#pragma unroll
                    for (int i = 0; i < DG_BN / 32; ++i) {
                        if (W_KMAJOR)
                            lfptx::tma_load_2d(a_dst + DG_A_BYTES + i * DG_BOX_BYTES, &map_w, bar, j0 + ks * DG_BK, tn * DG_BN + i * 32);
                        else
                            lfptx::tma_load_2d(a_dst + DG_A_BYTES + i * DG_BOX_BYTES, &map_w, bar, tn * DG_BN + i * 32,
                                           j0 + ks * DG_BK);
                    }
                }
                if (sh->abort_flag) break;
            }
            // after giving up: do not let the CTA exit under loads that are still landing
            if (sh->abort_flag) {
                const unsigned long long t0 = lfptx::globaltimer_ns();
                for (unsigned j = it > DG_STAGES ? it - DG_STAGES : 0; j < it; ++j) {
                    const unsigned bar = lfptx::smem_u32(&sh->full[j % DG_STAGES]);
                    while (!lfptx::mbar_try_wait(bar, (j / DG_STAGES) & 1u) && lfptx::globaltimer_ns() - t0 < 50000000ull) { }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer --------------------------------------------
        if (lane == 0) {
            const unsigned idesc = dg_idesc(W_KMAJOR);
            unsigned it = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    const unsigned st = it % DG_STAGES, use = it / DG_STAGES;
                    const unsigned p = it & 1u, p_use = it >> 1;
                    if (!dg_wait(lfptx::smem_u32(&sh->split_done[st]), use & 1u, P, sh)) { ok = false; break; }
                    if (p_use > 0 && !dg_wait(lfptx::smem_u32(&sh->acc_empty[p]), (p_use - 1) & 1u, P, sh)) { ok = false; break; }
                    lfptx::tc_fence_after();
                    const unsigned hi = lfptx::smem_u32(stages + (size_t)st * DG_STAGE_BYTES);
                    const unsigned lo = hi + DG_RAW_BYTES;
                    const unsigned d_tmem = tmem_base + p * (unsigned)DG_BN;
                    // the eight small products first, then the four large ones
#pragma unroll
                    for (int kk = 0; kk < DG_BK / 8; ++kk) {
                        dg_mma(d_tmem, dg_desc_kmajor(lo + kk * 32), dg_desc_w<W_KMAJOR>(hi + DG_A_BYTES, kk), idesc,
                               kk > 0 ? 1u : 0u);
                        dg_mma(d_tmem, dg_desc_kmajor(hi + kk * 32), dg_desc_w<W_KMAJOR>(lo + DG_A_BYTES, kk), idesc, 1u);
                    }
#pragma unroll
                    for (int kk = 0; kk < DG_BK / 8; ++kk)
                        dg_mma(d_tmem, dg_desc_kmajor(hi + kk * 32), dg_desc_w<W_KMAJOR>(hi + DG_A_BYTES, kk), idesc, 1u);
                    dg_commit(lfptx::smem_u32(&sh->empty[st]));
                    dg_commit(lfptx::smem_u32(&sh->acc_full[p]));
                }
            }
        }
    } else {
        // ---------------- operand split (hi/lo) and epilogue: warps 2..5 ----------------------
        const int tt = threadIdx.x - 64;
        const int quad = warp & 3;
        unsigned it = 0;
        bool ok = true;
        float acc[DG_BN];      // this thread's output row (sample), all 128 columns of the tile
        // add the finished stage `j` (accumulator j & 1) into the registers; first == overwrite
        auto drain = [&](unsigned j, bool first) -> bool {
            const unsigned p = j & 1u;
            if (!dg_wait(lfptx::smem_u32(&sh->acc_full[p]), (j >> 1) & 1u, P, sh)) return false;
            lfptx::tc_fence_after();
#pragma unroll
            for (int cchunk = 0; cchunk < DG_BN / 32; ++cchunk) {
                unsigned r[32];
                lfptx::tmem_ld32(tmem_base + ((unsigned)(quad * 32) << 16) + p * (unsigned)DG_BN + cchunk * 32, r);
#pragma unroll
                for (int v = 0; v < 32; ++v)
                    acc[cchunk * 32 + v] = first ? __uint_as_float(r[v]) : acc[cchunk * 32 + v] + __uint_as_float(r[v]);
            }
            lfptx::tc_fence_before();
            lfptx::mbar_arrive(lfptx::smem_u32(&sh->acc_empty[p]));
            return true;
        };
        for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
            const int tn = u % P.tiles_n, tm = (u / P.tiles_n) % P.tiles_m, sp = u / (P.tiles_n * P.tiles_m);
            for (int ks = 0; ks < n_k; ++ks, ++it) {
                const unsigned st = it % DG_STAGES, use = it / DG_STAGES;
                if (!dg_wait(lfptx::smem_u32(&sh->full[st]), use & 1u, P, sh)) { ok = false; break; }
                float4* raw = reinterpret_cast<float4*>(stages + (size_t)st * DG_STAGE_BYTES);
                float4* lo = reinterpret_cast<float4*>(stages + (size_t)st * DG_STAGE_BYTES + DG_RAW_BYTES);
#pragma unroll 4
                for (int i = 0; i < DG_RAW_BYTES / 16 / 128; ++i) {
                    const int idx = tt + i * 128;
                    const float4 v = raw[idx];
                    const float4 h = make_float4(dg_tf32_rn(v.x), dg_tf32_rn(v.y), dg_tf32_rn(v.z), dg_tf32_rn(v.w));
                    raw[idx] = h;
                    lo[idx] = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
                }
                // the tensor core reads shared memory through the async proxy
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                lfptx::mbar_arrive(lfptx::smem_u32(&sh->split_done[st]));
                if (ks > 0 && !drain(it - 1, ks == 1)) { ok = false; break; }
            }
            if (!ok) break;
            if (!drain(it - 1, n_k == 1)) { ok = false; break; }
            float* blk = epi + (warp - 2) * 32 * DG_EPI_LD;
            const int row0 = tm * DG_BM + quad * 32;
            const int sub_r = lane >> 3, sub_c = (lane & 7) * 4;
            float* out = P.partial + (size_t)sp * P.B * P.N;
#pragma unroll
            for (int cchunk = 0; cchunk < DG_BN / 32; ++cchunk) {
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<float4*>(blk + lane * DG_EPI_LD + 4 * v) =
                        make_float4(acc[cchunk * 32 + 4 * v], acc[cchunk * 32 + 4 * v + 1],
                                    acc[cchunk * 32 + 4 * v + 2], acc[cchunk * 32 + 4 * v + 3]);
                __syncwarp();
                const int col = tn * DG_BN + cchunk * 32 + sub_c;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = i * 4 + sub_r;
                    const float4 val = *reinterpret_cast<const float4*>(blk + rr * DG_EPI_LD + sub_c);
                    if (row0 + rr < P.B && col < P.N)
                        *reinterpret_cast<float4*>(out + (size_t)(row0 + rr) * P.N + col) = val;
                }
                __syncwarp();
            }
        }
    }

    lfptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        lfptx::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((unsigned)DG_TMEM_COLS)
                     : "memory");
    }
}

// ================================================================================================
// Two-SM form (more than 128 samples): a pair of CTAs (one thread-block cluster) works on
// 256 samples x 256 columns with tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 8).  Each CTA
// loads and splits only HALF of the W tile (128 columns), which the tensor cores of both CTAs
// read, so the shared-memory traffic per multiply-add falls; and the three jobs that share one
// set of warps in the kernel above -- splitting a stage, issuing its products, adding the
// finished stage into the running sums -- have warps of their own here, so they overlap:
//   warp 0       TMA producer: this CTA's 128 samples of D and its 128 columns of W per stage;
//   warp 1       leader CTA (cluster rank 0) only: issues the products for both CTAs;
//   warps 2-7    split this CTA's stage into hi/lo (high parts in place, the rest into a second ring);
//   warps 8-15   running sums of this CTA's 128 samples: a thread holds one sample and 128 of
//                the 256 columns in registers.  They need about 200 registers per thread and the
//                other warps few, so the warpgroups re-divide the register file at the start
//                (setmaxnreg: 2 x 128 threads x 48 + 2 x 128 threads x 208 = 512 x 128).
// Hand-offs across the pair: the splitting warps of both CTAs arrive on the leader's "split done"
// barrier, the leader's tcgen05.commit reaches the "raw slot free", "second-ring slot free" and
// "accumulator full" barriers of both CTAs, the summing warps of both arrive on the leader's
// "accumulator drained" barrier.
// Work is dealt by K block, not by tile: the tiles x K-blocks sequence is cut into one contiguous
// run per pair (runs differ by at most one block), so a pair may finish one tile's tail and
// start the next tile.  Every run segment inside a tile writes its partial sums to the slot
// given by its position among the segments of that tile; k_delta_finish / k_forward_finish add
// a tile's slots in that order, so the result does not depend on timing.
// Arithmetic per output element is that of the one-SM kernel above.
constexpr int DP_BN = 256;                               // columns of a pair tile (128 loaded per CTA)
constexpr int DP_BNH = DP_BN / 2;
constexpr int DP_B_BYTES = (DP_BNH / 32) * DG_BOX_BYTES; // 16 KiB (either operand form)
constexpr int DP_RAW_BYTES = DG_A_BYTES + DP_B_BYTES;    // 32 KiB per CTA and stage from TMA
// A stage lives in two rings.  Its raw tile (where the high parts then stand) holds a slot from the
// moment its load is issued until its products are done; what the split adds (remainders, or the
// 16-bit tiles) is only needed from the split on.  Four raw slots keep loads in the air behind the
// stage being worked on, and two slots of the second ring let the split of one stage run under the
// products of the one before.  With the hand-offs cheap (see dp_arrive_cluster) a stage of twelve
// TF32 instructions then takes about 2100 cycles, which is the rate the tensor cores issue them at.
constexpr int DP_RAW_SLOTS = 4, DP_LO_SLOTS = 2;
constexpr int DP_LO_BASE = DP_RAW_SLOTS * DP_RAW_BYTES;
constexpr int DP_RING_BYTES = (DP_RAW_SLOTS + DP_LO_SLOTS) * DP_RAW_BYTES;
constexpr int DP_THREADS = 512;                          // four warpgroups
constexpr int DP_SPLITTERS = 192;                        // warps 2-7
constexpr int DP_REGS_LAUNCH = 128, DP_REGS_SMALL = 48, DP_REGS_SUM = 208;
static_assert(2 * 128 * DP_REGS_SMALL + 2 * 128 * DP_REGS_SUM <= DP_THREADS * DP_REGS_LAUNCH,
              "the warpgroups' register shares must fit into what the CTA is launched with");
constexpr int DP_EPI_LD = 20;                            // 16 columns + padding
constexpr int DP_EPI_BYTES = 8 * 32 * DP_EPI_LD * 4;
constexpr size_t DP_SMEM_BYTES = (size_t)DP_RING_BYTES + DP_EPI_BYTES + 1024 + 256;
static_assert(DP_SMEM_BYTES <= 227 * 1024, "the two rings, the output staging and the barriers must fit one CTA");

struct DpShared {
    unsigned long long full[DP_RAW_SLOTS];      // this CTA's TMA data of the stage has landed
    unsigned long long raw_empty[DP_RAW_SLOTS]; // both: the products that read the raw slot are done
    unsigned long long split_done[DP_LO_SLOTS]; // leader: the stage is split in both CTAs (12 warp arrivals)
    unsigned long long lo_empty[DP_LO_SLOTS];   // both: the products that read the second-ring slot are done
    unsigned long long acc_full[2];            // both: stage accumulator p holds a finished stage
    unsigned long long acc_empty[2];           // leader: accumulator p drained by both CTAs (16 warp arrivals)
    unsigned tmem_base;
    volatile unsigned abort_flag;
};

__device__ __forceinline__ void dp_mma(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                       unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same instruction on 16-bit operands (here BF16 x BF16, sixteen values of the contraction index)
__device__ __forceinline__ void dp_mma16(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                         unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// MN-major 16-bit operand, 128-byte swizzle: 64 values along N per 128-byte row, eight K rows per
// 1024-byte atom (SBO), the next 64 columns one 32-row block (4 KiB) further (LBO).
__device__ __forceinline__ unsigned long long dp_desc_mnmajor16(unsigned smem_addr)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);
    d |= (unsigned long long)((4096u >> 4) & 0x3FFFu) << 16;
    d |= (unsigned long long)((1024u >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// BF16 operand of K step kk (sixteen values of the contraction index) of the W tile: part 0 = the
// high parts, part 1 = the remainders
template <bool W_KMAJOR>
__device__ __forceinline__ unsigned long long dp_desc_w16(unsigned tile16_addr, int part, int kk)
{
    return W_KMAJOR ? dg_desc_kmajor(tile16_addr + part * 64 + kk * 32)
                    : dp_desc_mnmajor16(tile16_addr + part * (DP_B_BYTES / 2) + kk * 2048);
}
// two fp32 values as BF16 (round to nearest, ties away from zero) in one word, the first in the low half
__device__ __forceinline__ unsigned dp_pack_bf16(float a, float b)
{
    return __byte_perm(__float_as_uint(a) + 0x8000u, __float_as_uint(b) + 0x8000u, 0x7632);
}
// arrive on the barrier at this offset in both CTAs once the tensor-core work issued so far is done
__device__ __forceinline__ void dp_commit_both(unsigned bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void dp_arrive_cluster(unsigned cluster_bar)
{
    // What the arriving warp wrote for the tensor cores has passed a proxy fence, what it read from
    // tensor memory a tcgen05 fence.  A release at cluster scope here (.release.cluster) was measured
    // at about 1300 cycles per hand-off, which then bounded the kernel at 3000 cycles per K stage.
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool dp_wait(unsigned bar, unsigned parity, const DgParams& P, DpShared* sh)
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
// The pair whose run contains block g when g_total blocks are cut into n_pairs runs
// [p * g_total / n_pairs, (p + 1) * g_total / n_pairs).
// (g_total * (n_pairs + 1) stays below 2^31: checked by the host before this tiling is chosen.)
__host__ __device__ __forceinline__ int dp_owner(int g, int g_total, int n_pairs)
{
    return ((g + 1) * n_pairs - 1) / g_total;
}
struct DpSegment {
    int tile;       // tm * tiles_n + tn
    int kb0, kb1;   // K blocks [kb0, kb1) of that tile
    int slot;       // which partial-sum slot of the tile this segment writes
};
// Next segment of the run [g, g1): advances g.  Every role of the kernel walks the same sequence.
__device__ __forceinline__ bool dp_next_segment(int& g, int g1, const DgParams& P, int pair, int n_pairs, DpSegment& sg)
{
    if (g >= g1) return false;
    sg.tile = g / P.kb_per_tile;
    sg.kb0 = g - sg.tile * P.kb_per_tile;
    const int left = g1 - g;
    sg.kb1 = left < P.kb_per_tile - sg.kb0 ? sg.kb0 + left : P.kb_per_tile;
    sg.slot = pair - dp_owner(sg.tile * P.kb_per_tile, P.g_total, n_pairs);
    g += sg.kb1 - sg.kb0;
    return true;
}
// fmt: operand format of the instruction kind (kind::tf32: 2 = TF32; kind::f16: 1 = BF16)
__device__ __forceinline__ unsigned dp_idesc(bool w_kmajor, unsigned fmt = 2u, int tile_m = 2 * DG_BM, int tile_n = DP_BN)
{
    unsigned d = 0;
    d |= 1u << 4;                             // fp32 accumulator
    d |= fmt << 7;                            // A
    d |= fmt << 10;                           // B
    d |= 0u << 15;                            // A is K-major
    d |= (w_kmajor ? 0u : 1u) << 16;          // B operand: K-major or MN-major
    d |= (unsigned)(tile_n >> 3) << 17;
    d |= (unsigned)(tile_m >> 4) << 24;
    return d;
}
// One product of a stage: a CTA pair's instruction (cta_group::2) or a single CTA's (cta_group::1);
// WIDE = false: TF32 operands, eight values of the contraction index; WIDE = true: BF16, sixteen.
template <bool PAIR, bool WIDE>
__device__ __forceinline__ void dp_product(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                           unsigned idesc, unsigned accumulate)
{
    if (PAIR) {
        if (WIDE) dp_mma16(d_tmem, a_desc, b_desc, idesc, accumulate);
        else dp_mma(d_tmem, a_desc, b_desc, idesc, accumulate);
    } else if (WIDE) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    } else {
        dg_mma(d_tmem, a_desc, b_desc, idesc, accumulate);
    }
}
// "everything issued so far is done" to a barrier of this CTA and, for a pair, of its peer
template <bool PAIR>
__device__ __forceinline__ void dp_commit(unsigned bar)
{
    if (PAIR) dp_commit_both(bar);
    else dg_commit(bar);
}
// 32 lanes x 64 consecutive fp32 columns of tensor memory as two loads in flight together
__device__ __forceinline__ void dp_tmem_ld64(unsigned taddr, unsigned (&r)[64])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]),
          "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]),
          "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]),
          "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr + 32u) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// What a splitting thread needs to place its pieces.  A raw stage is 256 rows of 128 bytes (the D
// tile, then the W tile), eight 16-byte pieces per row.  In round i a warp takes four rows of one
// group of eight rows -- its lanes 0-7, 8-15, 16-23, 24-31 the rows g, g + 4, g + 1, g + 5 of the
// group (g = 0 or 2) -- so that the 8-byte BF16 stores of a half-warp, which for rows g and g + 4 fall
// into opposite halves of the 128-byte lines, meet no bank twice.  A thread keeps its piece (tt & 7)
// and its row within the group, which all swizzle terms depend on; its row advances by 24 per round.
struct DpSplitPlace {
    unsigned idx0;        // 16-byte piece of round 0: row * 8 + (tt & 7)
    unsigned k_hi, k_lo;  // K-major tiles: byte offset in the BF16 row of the high parts / the remainders
    unsigned mn0, mn1;    // MN-major W: the same for an even / odd 32-column box (high parts)
};
__device__ __forceinline__ DpSplitPlace dp_split_place(int tt)
{
    DpSplitPlace pl;
    const unsigned p = tt & 7u, q = (tt >> 3) & 3u, w = (unsigned)tt >> 5;
    const unsigned sw = (w & 1u) * 2u + (q >> 1) + (q & 1u) * 4u;      // row within its group of eight = row & 7
    pl.idx0 = (8u * (w >> 1) + sw) * 8u + p;
    // K-major, 128-byte swizzle: piece p of a row holds K values 4c .. 4c+3, c = p ^ sw; as BF16 they
    // are eight bytes of piece c >> 1 (high parts) or 4 + (c >> 1) (remainders) of the BF16 row
    const unsigned ck = p ^ sw;
    pl.k_hi = (((ck >> 1) ^ sw) << 4) + (ck & 1u) * 8u;
    pl.k_lo = (((4u + (ck >> 1)) ^ sw) << 4) + (ck & 1u) * 8u;
    // MN-major W (32-byte swizzle atoms): piece p of K row k of a 32-column box holds columns
    // 4c .. 4c+3, c = p ^ ((k & 3) << 1); as BF16: K row k of a 64-column block, piece
    // ((box & 1) * 4 + (c >> 1)) ^ (k & 7), and k & 7 = sw here
    const unsigned cm = p ^ ((sw & 3u) << 1);
    pl.mn0 = (((cm >> 1) ^ sw) << 4) + (cm & 1u) * 8u;
    pl.mn1 = (((4u + (cm >> 1)) ^ sw) << 4) + (cm & 1u) * 8u;
    return pl;
}
// fp32 to TF32, round to nearest, ties away from zero (what cvt.rna.tf32.f32 gives), on the integer pipe
__device__ __forceinline__ float dp_tf32_rn(float x)
{
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}
// Round I (compile-time) of a thread's pieces: the TF32 high parts replace the raw values; the
// remainders go to the same place of the second-ring slot `lo`, or (CROSS_BF16) high parts and
// remainders go there as BF16.
template <bool W_KMAJOR, bool CROSS_BF16, int I>
__device__ __forceinline__ void dp_split_piece(float4* raw, float4* lo, const DpSplitPlace& pl, const float4 v)
{
    const unsigned idx = pl.idx0 + (unsigned)(I * DP_SPLITTERS), row = idx >> 3;     // rows 0 .. 127: D tile, 128 .. 255: W tile
    const float4 h = make_float4(dp_tf32_rn(v.x), dp_tf32_rn(v.y), dp_tf32_rn(v.z), dp_tf32_rn(v.w));
    raw[idx] = h;
    const float4 r = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
    if (!CROSS_BF16) {
        lo[idx] = r;
        return;
    }
    constexpr bool MAYBE_D = 24 * I < DG_BM, MAYBE_W = 23 + 24 * I >= DG_BM;
    unsigned off_h, off_r;
    if (W_KMAJOR || !MAYBE_W || (MAYBE_D && row < (unsigned)DG_BM)) {
        off_h = row * 128u + pl.k_hi;                // (the W tile follows the D tile at the same row pitch)
        off_r = row * 128u + pl.k_lo;
    } else {
        const unsigned box = (row - DG_BM) >> 5, k = row & 31u;
        off_h = (unsigned)DG_A_BYTES + (box >> 1) * 4096u + k * 128u + ((box & 1u) ? pl.mn1 : pl.mn0);
        off_r = off_h + (unsigned)(DP_B_BYTES / 2);
    }
    unsigned char* t16 = reinterpret_cast<unsigned char*>(lo);
    *reinterpret_cast<uint2*>(t16 + off_h) = make_uint2(dp_pack_bf16(h.x, h.y), dp_pack_bf16(h.z, h.w));
    *reinterpret_cast<uint2*>(t16 + off_r) = make_uint2(dp_pack_bf16(r.x, r.y), dp_pack_bf16(r.z, r.w));
}
// rounds I0 .. I0 + BATCH - 1: all loads first, then the arithmetic and the stores
template <bool W_KMAJOR, bool CROSS_BF16, int I0, int BATCH>
__device__ __forceinline__ void dp_split_batch(float4* raw, float4* lo, const DpSplitPlace& pl)
{
    float4 v[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) v[j] = raw[pl.idx0 + (unsigned)((I0 + j) * DP_SPLITTERS)];
    if constexpr (BATCH > 0) dp_split_piece<W_KMAJOR, CROSS_BF16, I0>(raw, lo, pl, v[0]);
    if constexpr (BATCH > 1) dp_split_piece<W_KMAJOR, CROSS_BF16, I0 + 1>(raw, lo, pl, v[1]);
    if constexpr (BATCH > 2) dp_split_piece<W_KMAJOR, CROSS_BF16, I0 + 2>(raw, lo, pl, v[2]);
    if constexpr (BATCH > 3) dp_split_piece<W_KMAJOR, CROSS_BF16, I0 + 3>(raw, lo, pl, v[3]);
    if constexpr (BATCH > 4) dp_split_piece<W_KMAJOR, CROSS_BF16, I0 + 4>(raw, lo, pl, v[4]);
}

// CROSS_BF16 = false: hi*hi + hi*lo + lo*hi in TF32 (twelve instructions per 32-wide K stage).
// CROSS_BF16 = true : hi*hi in TF32, the two cross terms in BF16 (eight instructions per stage): next to
//   the TF32 high parts the split warps write, where the fp32 remainders went, the high parts and the
//   remainders rounded to BF16 (K-major operands: both in one 128-byte row, high parts first; the
//   MN-major W tile: two tiles of 64-column blocks).  A cross term is below 2^-11 of its product, so
//   the 2^-9 of a BF16 rounding leaves about 2^-20 of the product.
// PAIR = false: the same kernel on single CTAs (no cluster): a CTA works alone on 128 samples x 128 columns
//   with cta_group::1 instructions (M = 128, N = 128) -- the warp-specialised form for 17 to 128 samples, where
//   a pair's second half would be empty; its summing warps hold 64 columns per thread.
template <bool W_KMAJOR, bool CROSS_BF16, bool PAIR>
__global__ void __launch_bounds__(DP_THREADS, 1)
k_delta_gemm_tc_pair(const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_w,
                     const DgParams P)
{
    extern __shared__ unsigned char dg_smem_raw[];
    // the same offsets in both CTAs: one descriptor addresses the shared memory of both
    unsigned char* stages = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(dg_smem_raw) + 1023u) & ~(uintptr_t)1023u);
    float* epi = reinterpret_cast<float*>(stages + (size_t)DP_RING_BYTES);
    DpShared* sh = reinterpret_cast<DpShared*>(stages + (size_t)DP_RING_BYTES + DP_EPI_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TILE_M = PAIR ? 2 * DG_BM : DG_BM, TILE_N = PAIR ? DP_BN : DP_BNH;   // tile of a pair / of a single CTA
    constexpr int SUM_COLS = TILE_N / 2;                    // columns a summing thread holds
    const unsigned rank = PAIR ? lfptx::cluster_ctarank() : 0u;
    const int pair = PAIR ? blockIdx.x >> 1 : blockIdx.x, n_pairs = PAIR ? gridDim.x >> 1 : gridDim.x;   // worker index and count
    const int g_begin = (int)((long long)P.g_total * pair / n_pairs), g_end = (int)((long long)P.g_total * (pair + 1) / n_pairs);
    DG_STAMP_ONCE(9);

    if (threadIdx.x == 0) {
        for (int i = 0; i < DP_RAW_SLOTS; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->raw_empty[i]), 1);
        }
        for (int i = 0; i < DP_LO_SLOTS; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->split_done[i]), (PAIR ? 2 : 1) * DP_SPLITTERS / 32);
            lfptx::mbar_init(lfptx::smem_u32(&sh->lo_empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            lfptx::mbar_init(lfptx::smem_u32(&sh->acc_full[i]), 1);
            lfptx::mbar_init(lfptx::smem_u32(&sh->acc_empty[i]), PAIR ? 16 : 8);
        }
        sh->abort_flag = 0u;
        lfptx::mbar_fence_init();
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(lfptx::smem_u32(&sh->tmem_base)), "r"((unsigned)(2 * TILE_N)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(lfptx::smem_u32(&sh->tmem_base)), "r"((unsigned)(2 * TILE_N)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    lfptx::tc_fence_before();
    __syncthreads();
    if (PAIR) lfptx::cluster_sync_all();   // the peer's barriers exist before anything can arrive on them
    lfptx::tc_fence_after();
    const unsigned tmem_base = sh->tmem_base;
    DG_STAMP_ONCE(10);

    if (warp < 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(DP_REGS_SMALL));
        if (warp == 0) {
            // ------------------------------ TMA producer (each CTA, its own halves) ------------
            if (lane == 0) {
                unsigned it = 0;
                bool ok = true;
                DpSegment sg;
                for (int g = g_begin; ok && dp_next_segment(g, g_end, P, pair, n_pairs, sg);) {
                    const int tn = sg.tile % P.tiles_n, tm = sg.tile / P.tiles_n;
                    const int j0 = sg.kb0 * DG_BK, n_k = sg.kb1 - sg.kb0;
                    const int row0 = tm * TILE_M + (int)rank * DG_BM;          // my samples
                    const int col0 = tn * TILE_N + (int)rank * DP_BNH;         // my columns of W
                    for (int ks = 0; ks < n_k; ++ks, ++it) {
                        const unsigned st = it % DP_RAW_SLOTS, use = it / DP_RAW_SLOTS;
                        if (use > 0 && !dp_wait(lfptx::smem_u32(&sh->raw_empty[st]), (use - 1) & 1u, P, sh)) { ok = false; break; }
                        DG_STAMP(0);
                        const unsigned bar = lfptx::smem_u32(&sh->full[st]);
                        lfptx::mbar_arrive_expect_tx(bar, DP_RAW_BYTES);
                        const unsigned a_dst = lfptx::smem_u32(stages + (size_t)st * DP_RAW_BYTES);
                        // boxes of 32 rows: the loads of one box are few at a time, several boxes go side by side
#pragma unroll
                        for (int i = 0; i < DG_BM / 32; ++i)
                            lfptx::tma_load_2d(a_dst + i * DG_BOX_BYTES, &map_d, bar, j0 + ks * DG_BK, row0 + i * 32);
#pragma unroll
                        for (int i = 0; i < DP_BNH / 32; ++i) {
                            if (W_KMAJOR)
                                lfptx::tma_load_2d(a_dst + DG_A_BYTES + i * DG_BOX_BYTES, &map_w, bar, j0 + ks * DG_BK, col0 + i * 32);
                            else
                                lfptx::tma_load_2d(a_dst + DG_A_BYTES + i * DG_BOX_BYTES, &map_w, bar, col0 + i * 32,
                                               j0 + ks * DG_BK);
                        }
                    }
                }
                // after giving up: do not let the CTA exit under loads that are still landing
                if (sh->abort_flag) {
                    const unsigned long long t0 = lfptx::globaltimer_ns();
                    for (unsigned j = it > DP_RAW_SLOTS ? it - DP_RAW_SLOTS : 0; j < it; ++j) {
                        const unsigned bar = lfptx::smem_u32(&sh->full[j % DP_RAW_SLOTS]);
                        while (!lfptx::mbar_try_wait(bar, (j / DP_RAW_SLOTS) & 1u) && lfptx::globaltimer_ns() - t0 < 50000000ull) { }
                    }
                }
            }
        } else if (warp == 1) {
            // ------------------------------ MMA issuer (leader CTA only) -----------------------
            if (lane == 0 && rank == 0) {
                const unsigned idesc = dp_idesc(W_KMAJOR, 2u, TILE_M, TILE_N), idesc16 = dp_idesc(W_KMAJOR, 1u, TILE_M, TILE_N);
                unsigned it = 0;
                bool ok = true;
                DpSegment sg;
                for (int g = g_begin; ok && dp_next_segment(g, g_end, P, pair, n_pairs, sg);) {
                    const int n_k = sg.kb1 - sg.kb0;
                    for (int ks = 0; ks < n_k; ++ks, ++it) {
                        // second-ring slot and stage accumulator alternate together
                        const unsigned st = it % DP_RAW_SLOTS, p = it & 1u, p_use = it >> 1;
                        if (!dp_wait(lfptx::smem_u32(&sh->split_done[p]), p_use & 1u, P, sh)) { ok = false; break; }
                        DG_STAMP(4);
                        if (p_use > 0 && !dp_wait(lfptx::smem_u32(&sh->acc_empty[p]), (p_use - 1) & 1u, P, sh)) { ok = false; break; }
                        DG_STAMP(5);
                        lfptx::tc_fence_after();
                        const unsigned hi = lfptx::smem_u32(stages + (size_t)st * DP_RAW_BYTES);
                        const unsigned lo = lfptx::smem_u32(stages + (size_t)DP_LO_BASE + (size_t)p * DP_RAW_BYTES);
                        const unsigned d_tmem = tmem_base + p * (unsigned)TILE_N;
                        // the small products first, then the four large ones
                        if (CROSS_BF16) {
#pragma unroll
                            for (int kk = 0; kk < DG_BK / 16; ++kk) {
                                dp_product<PAIR, true>(d_tmem, dg_desc_kmajor(lo + 64 + kk * 32), dp_desc_w16<W_KMAJOR>(lo + DG_A_BYTES, 0, kk),
                                                       idesc16, kk > 0 ? 1u : 0u);
                                dp_product<PAIR, true>(d_tmem, dg_desc_kmajor(lo + kk * 32), dp_desc_w16<W_KMAJOR>(lo + DG_A_BYTES, 1, kk),
                                                       idesc16, 1u);
                            }
                        } else {
#pragma unroll
                            for (int kk = 0; kk < DG_BK / 8; ++kk) {
                                dp_product<PAIR, false>(d_tmem, dg_desc_kmajor(lo + kk * 32), dg_desc_w<W_KMAJOR>(hi + DG_A_BYTES, kk), idesc,
                                                        kk > 0 ? 1u : 0u);
                                dp_product<PAIR, false>(d_tmem, dg_desc_kmajor(hi + kk * 32), dg_desc_w<W_KMAJOR>(lo + DG_A_BYTES, kk), idesc, 1u);
                            }
                        }
#pragma unroll
                        for (int kk = 0; kk < DG_BK / 8; ++kk)
                            dp_product<PAIR, false>(d_tmem, dg_desc_kmajor(hi + kk * 32), dg_desc_w<W_KMAJOR>(hi + DG_A_BYTES, kk), idesc, 1u);
                        dp_commit<PAIR>(lfptx::smem_u32(&sh->raw_empty[st]));
                        dp_commit<PAIR>(lfptx::smem_u32(&sh->lo_empty[p]));
                        dp_commit<PAIR>(lfptx::smem_u32(&sh->acc_full[p]));
                        DG_STAMP(6);
                    }
                }
            }
        } else {
            // ------------------------------ operand split (hi/lo): warps 2..7 ------------------
            const int tt = threadIdx.x - 64;
            const DpSplitPlace place = dp_split_place(tt);
            const unsigned leader_split_done0 = lfptx::map_to_cta(lfptx::smem_u32(&sh->split_done[0]), 0);
            unsigned it = 0;
            bool ok = true;
            DpSegment sg;
            for (int g = g_begin; ok && dp_next_segment(g, g_end, P, pair, n_pairs, sg);) {
                const int n_k = sg.kb1 - sg.kb0;
                for (int ks = 0; ks < n_k; ++ks, ++it) {
                    const unsigned st = it % DP_RAW_SLOTS, use = it / DP_RAW_SLOTS, ls = it & 1u, ls_use = it >> 1;
                    if (!dp_wait(lfptx::smem_u32(&sh->full[st]), use & 1u, P, sh)) { ok = false; break; }
                    if (tt == 0) DG_STAMP(1);
                    if (ls_use > 0 && !dp_wait(lfptx::smem_u32(&sh->lo_empty[ls]), (ls_use - 1) & 1u, P, sh)) { ok = false; break; }
                    if (tt == 0) DG_STAMP(2);
                    float4* raw = reinterpret_cast<float4*>(stages + (size_t)st * DP_RAW_BYTES);
                    float4* lo = reinterpret_cast<float4*>(stages + (size_t)DP_LO_BASE + (size_t)ls * DP_RAW_BYTES);
                    // 2048 16-byte pieces for 192 threads: ten rounds, a few loads in flight at a time, then 128 left
                    static_assert(DP_RAW_BYTES / 16 == 10 * DP_SPLITTERS + 128, "ten rounds and 128 pieces");
                    dp_split_batch<W_KMAJOR, CROSS_BF16, 0, 2>(raw, lo, place);
                    dp_split_batch<W_KMAJOR, CROSS_BF16, 2, 2>(raw, lo, place);
                    dp_split_batch<W_KMAJOR, CROSS_BF16, 4, 2>(raw, lo, place);
                    dp_split_batch<W_KMAJOR, CROSS_BF16, 6, 2>(raw, lo, place);
                    dp_split_batch<W_KMAJOR, CROSS_BF16, 8, 2>(raw, lo, place);
                    if (tt < 128) dp_split_batch<W_KMAJOR, CROSS_BF16, 10, 1>(raw, lo, place);
                    // the tensor cores (of both CTAs) read this shared memory through the async proxy
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (tt == 0) DG_STAMP(3);
                    if (lane == 0) dp_arrive_cluster(leader_split_done0 + ls * (unsigned)sizeof(unsigned long long));
                }
            }
        }
    } else {
        // ------------------------------ running sums and output: warps 8..15 -------------------
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(DP_REGS_SUM));
        const int quad = warp & 3;               // the TMEM lane quadrant this warp may read
        const int half = (warp - 8) >> 2;        // which half of the accumulator's columns
        const unsigned leader_acc_empty0 = lfptx::map_to_cta(lfptx::smem_u32(&sh->acc_empty[0]), 0);
        unsigned it = 0;
        bool ok = true;
        float acc[SUM_COLS];   // this thread's sample, its columns of the tile (128 for a pair, 64 for a single CTA)
        DpSegment sg;
        for (int g = g_begin; ok && dp_next_segment(g, g_end, P, pair, n_pairs, sg);) {
            const int tn = sg.tile % P.tiles_n, tm = sg.tile / P.tiles_n, sp = sg.slot;
            const int n_k = sg.kb1 - sg.kb0;
#pragma unroll
            for (int v = 0; v < SUM_COLS; ++v) acc[v] = 0.f;
            for (int ks = 0; ks < n_k; ++ks, ++it) {
                // add the finished stage (accumulator it & 1) into the registers
                const unsigned p = it & 1u;
                if (!dp_wait(lfptx::smem_u32(&sh->acc_full[p]), (it >> 1) & 1u, P, sh)) { ok = false; break; }
                if (threadIdx.x == 256) DG_STAMP(7);
                lfptx::tc_fence_after();
#pragma unroll
                for (int cchunk = 0; cchunk < SUM_COLS / 64; ++cchunk) {
                    unsigned r[64];
                    dp_tmem_ld64(tmem_base + ((unsigned)(quad * 32) << 16) + p * (unsigned)TILE_N + half * SUM_COLS + cchunk * 64, r);
#pragma unroll
                    for (int v = 0; v < 64; ++v)
                        acc[cchunk * 64 + v] += __uint_as_float(r[v]);
                }
                lfptx::tc_fence_before();
                __syncwarp();
                if (threadIdx.x == 256) DG_STAMP(8);
                if (lane == 0) dp_arrive_cluster(leader_acc_empty0 + p * (unsigned)sizeof(unsigned long long));
            }
            if (!ok) break;
            float* blk = epi + (warp - 8) * 32 * DP_EPI_LD;
            const int sub_r = lane >> 2, sub_c = (lane & 3) * 4;
            const int row0 = tm * TILE_M + (int)rank * DG_BM + quad * 32 + sub_r;
            const int col0 = tn * TILE_N + half * SUM_COLS + sub_c;
            // four rows per lane (row0 + 8 i), 16 columns per pass; constant offsets from one pointer per row
            float* out_row = P.partial + (size_t)sp * P.B * P.N + (size_t)row0 * P.N + col0;
            const size_t row_step = (size_t)8 * P.N;
#pragma unroll
            for (int cchunk = 0; cchunk < SUM_COLS / 16; ++cchunk) {
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    *reinterpret_cast<float4*>(blk + lane * DP_EPI_LD + 4 * v) =
                        make_float4(acc[cchunk * 16 + 4 * v], acc[cchunk * 16 + 4 * v + 1],
                                    acc[cchunk * 16 + 4 * v + 2], acc[cchunk * 16 + 4 * v + 3]);
                __syncwarp();
                if (col0 + cchunk * 16 < P.N) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 val = *reinterpret_cast<const float4*>(blk + (i * 8 + sub_r) * DP_EPI_LD + sub_c);
                        if (row0 + i * 8 < P.B)
                            *reinterpret_cast<float4*>(out_row + i * row_step + cchunk * 16) = val;
                    }
                }
                __syncwarp();
            }
        }
        DG_STAMP_ONCE(11);
    }

    // neither CTA may leave, or free tensor memory, while the other can still reach it
    lfptx::tc_fence_before();
    __syncthreads();
    if (PAIR) lfptx::cluster_sync_all();
    DG_STAMP_ONCE(12);
    if (warp == 1) {
        lfptx::tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((unsigned)(2 * TILE_N)) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((unsigned)(2 * TILE_N)) : "memory");
    }
}

// How many partial-sum slots hold a contribution to output element i (float4 index into [B][N]).
// One-SM kernel: the same number of K splits everywhere.  Two-SM kernel (n_pairs > 0): as many as
// there are run segments in the element's tile.
struct DgSlots {
    int splits;
    int n_pairs, tiles_n, kb_per_tile, row4;   // row4 = N / 4; n_pairs: workers (pairs or single CTAs) of the run-dealing kernel
    int g_total;
    int tile_m, tile_n;                        // its tile: 256 x 256 for pairs, 128 x 128 for single CTAs
};
// slots that hold a contribution to the output elements of sample b, columns n .. n+3
__device__ __forceinline__ int dg_slot_count(const DgSlots& S, int b, int n)
{
    if (S.n_pairs == 0) return S.splits;
    const int g0 = ((b / S.tile_m) * S.tiles_n + n / S.tile_n) * S.kb_per_tile;
    return dp_owner(g0 + S.kb_per_tile - 1, S.g_total, S.n_pairs) - dp_owner(g0, S.g_total, S.n_pairs) + 1;
}
// the sum of an element's slots, in slot order; the loads go out four at a time
__device__ __forceinline__ float4 dg_slot_sum(const float4* __restrict__ p, size_t slot_stride, int splits)
{
    float4 s = __ldcg(p);
    int sp = 1;
    for (; sp + 4 <= splits; sp += 4) {
        const float4 t0 = __ldcg(p + (size_t)sp * slot_stride), t1 = __ldcg(p + (size_t)(sp + 1) * slot_stride);
        const float4 t2 = __ldcg(p + (size_t)(sp + 2) * slot_stride), t3 = __ldcg(p + (size_t)(sp + 3) * slot_stride);
        s.x += t0.x; s.y += t0.y; s.z += t0.z; s.w += t0.w;
        s.x += t1.x; s.y += t1.y; s.z += t1.z; s.w += t1.w;
        s.x += t2.x; s.y += t2.y; s.z += t2.z; s.w += t2.w;
        s.x += t3.x; s.y += t3.y; s.z += t3.z; s.w += t3.w;
    }
    for (; sp < splits; ++sp) {
        const float4 t = __ldcg(p + (size_t)sp * slot_stride);
        s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
    }
    return s;
}

// grid of the finish kernels: x = blocks of 256 float4 along a row of the output, y = sample
// delta^l = (sum over the partial-sum slots, in slot order) * sigma'(z^l), sigma' = a (1 - a)
__global__ void __launch_bounds__(256)
k_delta_finish(const float* __restrict__ partial, const float* __restrict__ a_l, float* __restrict__ delta_l,
               size_t n4, const DgSlots S, int act)
{
    const int c4 = blockIdx.x * blockDim.x + threadIdx.x;
    if (c4 >= S.row4) return;
    const int B = (int)(n4 / (size_t)S.row4);
    for (int b = blockIdx.y; b < B; b += gridDim.y) {       // (the grid holds at most 65535 samples)
        const size_t i = (size_t)b * S.row4 + c4;
        const float4 s = dg_slot_sum(reinterpret_cast<const float4*>(partial) + i, n4, dg_slot_count(S, b, 4 * c4));
        const float4 av = reinterpret_cast<const float4*>(a_l)[i];
        reinterpret_cast<float4*>(delta_l)[i] = make_float4(s.x * lf_act_prime(av.x, act), s.y * lf_act_prime(av.y, act),
                                                            s.z * lf_act_prime(av.z, act), s.w * lf_act_prime(av.w, act));
    }
}

// forward: z^l = (sum over the partial-sum slots) + b^l ; a^l = sigma(z^l)
__global__ void __launch_bounds__(256)
k_forward_finish(const float* __restrict__ partial, const float* __restrict__ b_l, float* __restrict__ z_l,
                 float* __restrict__ a_l, size_t n4, const DgSlots S, int act)
{
    const int c4 = blockIdx.x * blockDim.x + threadIdx.x;
    if (c4 >= S.row4) return;
    const int B = (int)(n4 / (size_t)S.row4);
    const float4 bb = reinterpret_cast<const float4*>(b_l)[c4];
    for (int b = blockIdx.y; b < B; b += gridDim.y) {
        const size_t i = (size_t)b * S.row4 + c4;
        float4 s = dg_slot_sum(reinterpret_cast<const float4*>(partial) + i, n4, dg_slot_count(S, b, 4 * c4));
        s.x += bb.x; s.y += bb.y; s.z += bb.z; s.w += bb.w;
        reinterpret_cast<float4*>(z_l)[i] = s;
        reinterpret_cast<float4*>(a_l)[i] = make_float4(lf_act(s.x, act), lf_act(s.y, act), lf_act(s.z, act), lf_act(s.w, act));
    }
}

typedef CUresult (*dg_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

dg_encode_fn dg_get_encode()
{
    static dg_encode_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<dg_encode_fn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

struct DgPlan {
    int tiles_m, tiles_n, splits, k_per_split;
    int pairs, kb_per_tile;      // run-dealing kernel (pairs > 0): launched pairs (or single CTAs) and K blocks per tile
    int g_total;
    int tile_m, tile_n;          // its tile (0: the plain one-SM kernel's fixed 128 x 128)
    bool solo;                   // run-dealing kernel on single CTAs
};

// One contraction out[B][Nc] = lhs[B][K] x W: Nc output columns, contraction length K.  Eq. bp2 of
// layer l has Nc = n_l, K = n_{l+1}; Eq. z of layer l has Nc = n_l, K = n_{l-1}.
DgPlan dg_plan(const lf_ctx* c, int Nc, int K)
{
    DgPlan p = {};
    p.tiles_m = (c->B + DG_BM - 1) / DG_BM;
    p.tiles_n = (Nc + DG_BN - 1) / DG_BN;
    int s = c->sm_count / (p.tiles_m * p.tiles_n);
    if (s < 1) s = 1;
    if (s > 8) s = 8;
    const int kb = (K + DG_BK - 1) / DG_BK;               // K blocks in all
    if (s > kb) s = kb;
    const int kb_per = (kb + s - 1) / s;
    p.splits = (kb + kb_per - 1) / kb_per;                 // no empty split
    p.k_per_split = kb_per * DG_BK;
    return p;
}

// Largest number of CTA pairs of the two-SM kernels that can be resident at once (0: unusable).
// Queried once per device; also opts the kernels in to their dynamic shared memory.
int dp_max_pairs(const lf_ctx* c)
{
    static int cached_dev = -1, cached = 0;
    if (cached_dev == c->device) return cached;
    int n = 0;
    if ((size_t)c->smem_optin >= DP_SMEM_BYTES &&
        cudaFuncSetAttribute(k_delta_gemm_tc_pair<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)DP_SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(k_delta_gemm_tc_pair<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)DP_SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(k_delta_gemm_tc_pair<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)DP_SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(k_delta_gemm_tc_pair<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)DP_SMEM_BYTES) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        cfg.gridDim = dim3(2 * 16); cfg.blockDim = dim3(DP_THREADS); cfg.dynamicSmemBytes = DP_SMEM_BYTES;
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n0 = 0, n1 = 0, n2 = 0, n3 = 0;
        if (cudaOccupancyMaxActiveClusters(&n0, k_delta_gemm_tc_pair<false, false, true>, &cfg) == cudaSuccess &&
            cudaOccupancyMaxActiveClusters(&n1, k_delta_gemm_tc_pair<true, false, true>, &cfg) == cudaSuccess &&
            cudaOccupancyMaxActiveClusters(&n2, k_delta_gemm_tc_pair<false, true, true>, &cfg) == cudaSuccess &&
            cudaOccupancyMaxActiveClusters(&n3, k_delta_gemm_tc_pair<true, true, true>, &cfg) == cudaSuccess) {
            n = n0 < n1 ? n0 : n1;
            if (n2 < n) n = n2;
            if (n3 < n) n = n3;
        }
    }
    cudaGetLastError();
    cached_dev = c->device; cached = n;
    return n;
}

// Largest number of CTAs of the single-CTA form of that kernel that can be resident at once (0: unusable).
int dp_max_solo(const lf_ctx* c)
{
    static int cached_dev = -1, cached = 0;
    if (cached_dev == c->device) return cached;
    int n = 0;
    if ((size_t)c->smem_optin >= DP_SMEM_BYTES &&
        cudaFuncSetAttribute(k_delta_gemm_tc_pair<false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)DP_SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(k_delta_gemm_tc_pair<true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)DP_SMEM_BYTES) == cudaSuccess) {
        int n0 = 0, n1 = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n0, k_delta_gemm_tc_pair<false, false, false>, DP_THREADS,
                                                          DP_SMEM_BYTES) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n1, k_delta_gemm_tc_pair<true, false, false>, DP_THREADS,
                                                          DP_SMEM_BYTES) == cudaSuccess)
            n = (n0 < n1 ? n0 : n1) > 0 ? c->sm_count : 0;      // one CTA per SM: each holds most of its shared memory
    }
    cudaGetLastError();
    cached_dev = c->device; cached = n;
    return n;
}

// The two-SM kernels pay off once a pair's 256 samples are more than half filled.
bool dp_use_pairs(const lf_ctx* c, int Nc, int K);

// Two-SM kernel: tiles x K-blocks cut into one contiguous run per pair; `splits` becomes the
// largest number of run segments (= partial-sum slots) any tile has.
DgPlan dp_plan(const lf_ctx* c, int Nc, int K, int max_pairs, bool solo = false)
{
    DgPlan p = {};
    p.solo = solo;
    p.tile_m = solo ? DG_BM : 2 * DG_BM; p.tile_n = solo ? DP_BNH : DP_BN;
    p.tiles_m = (c->B + p.tile_m - 1) / p.tile_m;
    p.tiles_n = (Nc + p.tile_n - 1) / p.tile_n;
    p.kb_per_tile = (K + DG_BK - 1) / DG_BK;
    p.k_per_split = p.kb_per_tile * DG_BK;
    const int tiles = p.tiles_m * p.tiles_n;
    const long long g_total = (long long)tiles * p.kb_per_tile;
    if (g_total * (max_pairs + 1) >= (1ll << 31)) return p;      // pairs == 0: not usable at this size
    p.g_total = (int)g_total;
    // no run shorter than four K blocks: below that the per-run set-up and output outweigh the balance
    const int by_length = p.g_total / 4 > 0 ? p.g_total / 4 : 1;
    p.pairs = by_length < max_pairs ? by_length : max_pairs;
    p.splits = 1;
    for (int t = 0; t < tiles; ++t) {
        const int g0 = t * p.kb_per_tile;
        const int n = dp_owner(g0 + p.kb_per_tile - 1, p.g_total, p.pairs) - dp_owner(g0, p.g_total, p.pairs) + 1;
        if (n > p.splits) p.splits = n;
    }
    return p;
}

// could the two-SM kernel be chosen for this shape (whatever LF_OPT_TC_TILING says)?
// Pairs need more than 128 samples: with fewer, their second CTA's samples are empty, and the
// warp-specialised kernel on single CTAs (below) is ahead at every width measured (N = 8192, 17 to 128
// samples, forward / backward per layer: 122-128 / 161-171 us against the pairs' 138-146 / 175-188).
// Narrow layers are launch-latency-bound: the lighter one-SM kernel is faster there.
bool dp_shape_fits_pairs(const lf_ctx* c, int Nc, int K)
{
    return c->B > DG_BM && Nc >= 512 && K >= 512 && dp_max_pairs(c) > 0;
}

bool dp_use_pairs(const lf_ctx* c, int Nc, int K)
{
    return c->tc_pair_kernels && dp_shape_fits_pairs(c, Nc, K) && dp_plan(c, Nc, K, dp_max_pairs(c)).pairs > 0;
}

// The warp-specialised kernel on single CTAs, where pairs do not apply: for layers of at least
// DP_SOLO_MIN_WIDTH.  Measured per layer (forward / backward, 17 to 128 samples) against the plain
// one-SM kernel: N = 2048 and 3072 level, N = 4096: 41-45 / 53-59 against 48-50 / 59-63 us,
// N = 5120: 57-60 / 74-81 against 73-75 / 88-93 us.  With fewer than 17 samples only the forward pass comes here.
#ifndef DP_SOLO_MIN_WIDTH
#define DP_SOLO_MIN_WIDTH 4096
#endif
bool dp_shape_fits_solo(const lf_ctx* c, int Nc, int K)
{
    return Nc >= DP_SOLO_MIN_WIDTH && K >= DP_SOLO_MIN_WIDTH && dp_max_solo(c) > 0;
}
bool dp_use_solo(const lf_ctx* c, int Nc, int K)
{
    return !dp_use_pairs(c, Nc, K) && dp_shape_fits_solo(c, Nc, K) && dp_plan(c, Nc, K, dp_max_solo(c), true).pairs > 0;
}

// floats of partial-sum scratch one contraction of this shape may need: [splits][B][Nc] of
// whichever tiling has more splits
size_t dg_partial_floats(const lf_ctx* c, int Nc, int K)
{
    int splits = dg_plan(c, Nc, K).splits;
    if (dp_shape_fits_pairs(c, Nc, K)) {
        const int s2 = dp_plan(c, Nc, K, dp_max_pairs(c)).splits;
        if (s2 > splits) splits = s2;
    }
    if (dp_shape_fits_solo(c, Nc, K)) {
        const int s3 = dp_plan(c, Nc, K, dp_max_solo(c), true).splits;
        if (s3 > splits) splits = s3;
    }
    return (size_t)splits * c->B * Nc;
}

}  // namespace

size_t lf_delta_tc_scratch_bytes(const lf_ctx* c)
{
    if (c->B < 2) return 0;
    // the largest need over every contraction of a pass: Eq. z of layers 1..L, Eq. bp2 of layers 1..L-1
    size_t floats = 0;
    for (int l = 1; l <= c->L; ++l) {
        size_t f = dg_partial_floats(c, c->width[l], c->width[l - 1]);
        if (f > floats) floats = f;
        if (l < c->L) {
            f = dg_partial_floats(c, c->width[l], c->width[l + 1]);
            if (f > floats) floats = f;
        }
    }
    return floats * sizeof(float);
}

bool lf_delta_tc_supported(const lf_ctx* c)
{
    if (c->B < 2 || !c->dg_partial) return false;
    if ((size_t)c->smem_optin < DG_SMEM_BYTES) return false;
    if (!dg_get_encode()) return false;
    static int attr_dev = -1;
    if (attr_dev != c->device) {
        if (cudaFuncSetAttribute(k_delta_gemm_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)DG_SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(k_delta_gemm_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)DG_SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        attr_dev = c->device;
    }
    dp_max_pairs(c);
    dp_max_solo(c);
    return true;
}

static DgSlots dg_slots(int Nc, const DgPlan& pl)
{
    DgSlots S = {};
    S.splits = pl.splits; S.n_pairs = pl.pairs; S.tiles_n = pl.tiles_n; S.kb_per_tile = pl.kb_per_tile;
    S.row4 = Nc / 4; S.g_total = pl.g_total;
    S.tile_m = pl.tile_m; S.tile_n = pl.tile_n;
    return S;
}

// Encode the two operand maps and launch one contraction out[B][Nc] = lhs[B][K] x W into
// c->dg_partial.  W is [Nc][K] (w_kmajor: row n holds the K values it is contracted over, Eq. z) or
// [K][Nc] (Eq. bp2: the transposed product read from the same row-major matrix).
static int dg_launch(lf_ctx* c, const float* lhs, const float* w_mat, bool w_kmajor, bool cross_bf16, int Nc, int K,
                     cudaStream_t s, DgPlan* plan_out)
{
    alignas(64) CUtensorMap map_d, map_w;
    {
        cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)c->B};
        cuuint64_t strides[1] = {(cuuint64_t)K * 4};
        cuuint32_t box[2] = {32, 32};                        // 32 values of j x 32 samples
        cuuint32_t estr[2] = {1, 1};
        if (dg_get_encode()(&map_d, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(lhs), dims, strides,
                            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            c->last_cuda_error = (int)cudaErrorInvalidValue;
            return LF_ECUDA;
        }
    }
    {
        const int inner = w_kmajor ? K : Nc, outer = w_kmajor ? Nc : K;
        cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
        cuuint64_t strides[1] = {(cuuint64_t)inner * 4};
        cuuint32_t box_mn[2] = {32, (cuuint32_t)DG_BK};      // 32 columns n x 32 rows j
        cuuint32_t box_k[2] = {32, 32};                      // 32 values of j x 32 rows n
        cuuint32_t estr[2] = {1, 1};
        if (dg_get_encode()(&map_w, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(w_mat), dims, strides,
                            w_kmajor ? box_k : box_mn, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            w_kmajor ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            c->last_cuda_error = (int)cudaErrorInvalidValue;
            return LF_ECUDA;
        }
    }
    const bool pairs = dp_use_pairs(c, Nc, K);
    const bool solo = !pairs && dp_use_solo(c, Nc, K);
    const DgPlan pl = pairs ? dp_plan(c, Nc, K, dp_max_pairs(c)) : solo ? dp_plan(c, Nc, K, dp_max_solo(c), true) : dg_plan(c, Nc, K);
    if ((size_t)pl.splits * c->B * Nc > dg_partial_floats(c, Nc, K)) return LF_ERESOURCE;   // cannot happen: same plans
    DgParams P;
    P.N = Nc; P.B = c->B;
    P.tiles_m = pl.tiles_m; P.tiles_n = pl.tiles_n; P.splits = pl.splits; P.k_per_split = pl.k_per_split;
    P.kb_per_tile = pl.kb_per_tile; P.g_total = pl.g_total;
    P.partial = c->dg_partial;
    P.status = c->status_dev;
    P.budget_ns = (unsigned long long)c->wait_budget_us * 1000ull;
    const int units = pl.tiles_m * pl.tiles_n * pl.splits;
    if (pairs) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        cfg.gridDim = dim3(2 * pl.pairs);
        cfg.blockDim = dim3(DP_THREADS); cfg.dynamicSmemBytes = DP_SMEM_BYTES; cfg.stream = s;
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        if (w_kmajor && cross_bf16)
            LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_delta_gemm_tc_pair<true, true, true>, map_d, map_w, P));
        else if (w_kmajor)
            LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_delta_gemm_tc_pair<true, false, true>, map_d, map_w, P));
        else if (cross_bf16)
            LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_delta_gemm_tc_pair<false, true, true>, map_d, map_w, P));
        else
            LF_CUDA_TRY(c, cudaLaunchKernelEx(&cfg, k_delta_gemm_tc_pair<false, false, true>, map_d, map_w, P));
        c->stats.delta_tiling = LF_TC_TILING_TWO_SM;
        *plan_out = pl;
        return LF_OK;
    }
    c->stats.delta_tiling = LF_TC_TILING_ONE_SM;
    if (solo) {      // the warp-specialised kernel on single CTAs (the BF16 cross-term form is for pairs)
        if (w_kmajor)
            k_delta_gemm_tc_pair<true, false, false><<<pl.pairs, DP_THREADS, DP_SMEM_BYTES, s>>>(map_d, map_w, P);
        else
            k_delta_gemm_tc_pair<false, false, false><<<pl.pairs, DP_THREADS, DP_SMEM_BYTES, s>>>(map_d, map_w, P);
        LF_CUDA_TRY(c, cudaGetLastError());
        *plan_out = pl;
        return LF_OK;
    }
    const int grid = units < c->sm_count ? units : c->sm_count;
    if (w_kmajor)
        k_delta_gemm_tc<true><<<grid, DG_THREADS, DG_SMEM_BYTES, s>>>(map_d, map_w, P);
    else
        k_delta_gemm_tc<false><<<grid, DG_THREADS, DG_SMEM_BYTES, s>>>(map_d, map_w, P);
    LF_CUDA_TRY(c, cudaGetLastError());
    *plan_out = pl;
    return LF_OK;
}

int lf_delta_gemm_tc(lf_ctx* c, const float* w_up, const float* delta_up, const float* a_l, float* delta_l,
                     int n_up, int n_l, int math, cudaStream_t s, int* launches)
{
    // w_up = w^{l+1} is n_up x n_l; out[b][k] = sum_j delta_up[b][j] w_up[j][k]
    DgPlan pl;
    int rc = dg_launch(c, delta_up, w_up, false, math == LF_DELTA_MATH_TF32_BF16, n_l, n_up, s, &pl);
    if (rc != LF_OK) return rc;
    const size_t n4 = (size_t)c->B * n_l / 4;
    k_delta_finish<<<dim3((unsigned)((n_l / 4 + 255) / 256), (unsigned)(c->B < 65535 ? c->B : 65535)), 256, 0, s>>>(c->dg_partial, a_l, delta_l, n4,
                                                                                       dg_slots(n_l, pl), c->opt_act);
    LF_CUDA_TRY(c, cudaGetLastError());
    *launches += 2;
    return LF_OK;
}

int lf_forward_gemm_tc(lf_ctx* c, const float* w_l, const float* b_l, const float* a_prev, float* z_l, float* a_l,
                       int n_out, int n_in, int math, cudaStream_t s, int* launches)
{
    // w_l is n_out x n_in; out[b][j] = sum_k a_prev[b][k] w_l[j][k]
    DgPlan pl;
    int rc = dg_launch(c, a_prev, w_l, true, math == LF_DELTA_MATH_TF32_BF16, n_out, n_in, s, &pl);
    if (rc != LF_OK) return rc;
    const size_t n4 = (size_t)c->B * n_out / 4;
    k_forward_finish<<<dim3((unsigned)((n_out / 4 + 255) / 256), (unsigned)(c->B < 65535 ? c->B : 65535)), 256, 0, s>>>(c->dg_partial, b_l, z_l, a_l, n4,
                                                                                           dg_slots(n_out, pl), c->opt_act);
    LF_CUDA_TRY(c, cudaGetLastError());
    *launches += 2;
    return LF_OK;
}
