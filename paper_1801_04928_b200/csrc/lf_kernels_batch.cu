// Mini-batch (B > 1) kernels in fp32 on the CUDA cores.  With B samples as columns, Eq. z,
// Eq. bp2 and Eq. bp4 each become one dense N x N x B contraction per layer:
//     forward : Z[b][j]  = sum_k A[b][k]  W[j][k] + bias[j],  A' = sigma(Z)
//     delta   : D'[b][k] = (sum_j D[b][j] W[j][k]) * a[b][k] (1 - a[b][k])
//     grad_w  : G[j][k]  = sum_b D[b][j]  A[b][k]
// One shared-memory tiled kernel serves all three; the operand orientation (which index is
// contiguous in memory) and the epilogue are template parameters.
#include "lf_internal.h"

namespace {

constexpr int BM = 64, BN = 64, BK = 16, PAD = 4;

enum { EPI_PLAIN = 0, EPI_FORWARD = 1, EPI_DELTA = 2 };

// C[m][n] = sum_k A(m,k) Bm(k,n).
//   A_KMAJOR: A(m,k) = A[m*lda + k]   else A(m,k) = A[k*lda + m]
//   B_KMAJOR: Bm(k,n) = Bm[n*ldb + k] else Bm(k,n) = Bm[k*ldb + n]
// The contiguous extent of every operand (and Nn, ldc) must be a multiple of 4.
template <bool A_KMAJOR, bool B_KMAJOR, int EPI>
__global__ void __launch_bounds__(256)
k_gemm_simt(const float* __restrict__ A, const float* __restrict__ Bm, float* __restrict__ C,
            float* __restrict__ C2, const float* __restrict__ aux, int M, int Nn, int K, int lda,
            int ldb, int ldc, float eta, int act)
{
    __shared__ __align__(16) float As[BK][BM + PAD];
    __shared__ __align__(16) float Bs[BK][BN + PAD];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    // EPI_PLAIN with a weight matrix to update: fetch its values now, they are needed last
    float4 wsub[4];
    if (EPI == EPI_PLAIN && aux && n0 + tx * 4 < Nn) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (m0 + ty * 4 + i < M)
                wsub[i] = *reinterpret_cast<const float4*>(aux + (size_t)(m0 + ty * 4 + i) * ldc + n0 + tx * 4);
    }

    for (int k0 = 0; k0 < K; k0 += BK) {
        // ---- stage the A tile as As[k][m]
        if (A_KMAJOR) {
            int m = tid >> 2, kq = (tid & 3) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m0 + m < M && k0 + kq < K)
                v = *reinterpret_cast<const float4*>(A + (size_t)(m0 + m) * lda + k0 + kq);
            As[kq + 0][m] = v.x; As[kq + 1][m] = v.y; As[kq + 2][m] = v.z; As[kq + 3][m] = v.w;
        } else {
            int kk = tid >> 4, mq = (tid & 15) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < K && m0 + mq < M)
                v = *reinterpret_cast<const float4*>(A + (size_t)(k0 + kk) * lda + m0 + mq);
            *reinterpret_cast<float4*>(&As[kk][mq]) = v;
        }
        // ---- stage the B tile as Bs[k][n]
        if (B_KMAJOR) {
            int n = tid >> 2, kq = (tid & 3) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (n0 + n < Nn && k0 + kq < K)
                v = *reinterpret_cast<const float4*>(Bm + (size_t)(n0 + n) * ldb + k0 + kq);
            Bs[kq + 0][n] = v.x; Bs[kq + 1][n] = v.y; Bs[kq + 2][n] = v.z; Bs[kq + 3][n] = v.w;
        } else {
            int kk = tid >> 4, nq = (tid & 15) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < K && n0 + nq < Nn)
                v = *reinterpret_cast<const float4*>(Bm + (size_t)(k0 + kk) * ldb + n0 + nq);
            *reinterpret_cast<float4*>(&Bs[kk][nq]) = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            float ar[4] = {av.x, av.y, av.z, av.w};
            float br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
        __syncthreads();
    }

    const int n = n0 + tx * 4;
    if (n >= Nn) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= M) continue;
        float4 r = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        size_t off = (size_t)m * ldc + n;
        if (EPI == EPI_FORWARD) {
            float4 bb = *reinterpret_cast<const float4*>(aux + n);
            r.x += bb.x; r.y += bb.y; r.z += bb.z; r.w += bb.w;
            *reinterpret_cast<float4*>(C + off) = r;                       // z
            *reinterpret_cast<float4*>(C2 + off) = make_float4(lf_act(r.x, act), lf_act(r.y, act),
                                                               lf_act(r.z, act), lf_act(r.w, act));
        } else if (EPI == EPI_DELTA) {
            float4 av = *reinterpret_cast<const float4*>(aux + off);
            r.x *= lf_act_prime(av.x, act); r.y *= lf_act_prime(av.y, act);
            r.z *= lf_act_prime(av.z, act); r.w *= lf_act_prime(av.w, act);
            *reinterpret_cast<float4*>(C + off) = r;
        } else {
            // EPI_PLAIN: the contraction itself, or (aux = the weight matrix) aux - eta * it
            if (aux) r = lf_sgd_apply4(eta, wsub[i], r);
            *reinterpret_cast<float4*>(C + off) = r;
        }
    }
}

// Eq. bp3 for a mini-batch: gb_j = sum_b delta_bj.  A CTA owns 32 columns; warp w adds the
// samples w, w+8, ... (lanes = columns, 128-byte rows), then the eight warp sums are added in
// warp order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256)
k_grad_b_colsum(const float* __restrict__ delta_l, float* __restrict__ gb_l, int N, int B)
{
    __shared__ float part[8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * 32 + lane;
    float s0 = 0.f, s1 = 0.f;
    if (j < N) {
        int b = warp;
        for (; b + 8 < B; b += 16) {
            s0 += delta_l[(size_t)b * N + j];
            s1 += delta_l[(size_t)(b + 8) * N + j];
        }
        if (b < B) s0 += delta_l[(size_t)b * N + j];
    }
    part[warp][lane] = s0 + s1;
    __syncthreads();
    if (warp == 0 && j < N) {
        float s = part[0][lane];
#pragma unroll
        for (int q = 1; q < 8; ++q) s += part[q][lane];
        gb_l[j] = s;
    }
}

inline dim3 gemm_grid(int M, int Nn) { return dim3((Nn + BN - 1) / BN, (M + BM - 1) / BM); }

}  // namespace

cudaError_t lfk_forward_gemm(const float* w_l, const float* b_l, const float* a_prev,
                             float* z_l, float* a_l, int n_out, int n_in, int B, int act, cudaStream_t s)
{
    // M = B (samples), Nn = n_out (neuron j), K = n_in (neuron k of the layer below)
    k_gemm_simt<true, true, EPI_FORWARD><<<gemm_grid(B, n_out), 256, 0, s>>>(
        a_prev, w_l, z_l, a_l, b_l, B, n_out, n_in, n_in, n_in, n_out, 0.f, act);
    return cudaGetLastError();
}


namespace {

// ---- Eq. bp2 for a handful of samples (B <= 16) --------------------------------------------------
// With so few samples the contraction is a batched matrix-vector product: w^{l+1} is read once, at the
// memory rate, and every loaded weight is used B times from registers (4B fused multiply-adds per
// 16 bytes).  Tiles of tensor-core size would spend their time staging a nearly empty operand.
//   grid = column strips (128 columns) x row chunks, sized to one wave of resident CTAs.  A CTA of
//   eight warps walks the rows of its chunk (warp q: rows q, q+8, ...), each lane four columns and BT
//   running sums of them.  Every thread prefetches its own 16 bytes of the next SB_DEPTH rows with
//   cp.async into a ring slot only it reads, so the loads in flight cost no registers and need no
//   barrier.  The delta values of 256 rows at a time sit in shared memory as float4 over four
//   samples, so one broadcast 128-bit load feeds four samples.
//   Partial sums go to scratch [chunks][B][n_l]; the last CTA of a strip to finish adds them in chunk
//   order (a fixed order: results are reproducible), applies sigma' and writes delta^l.
constexpr int SB_WARPS = 8, SB_THREADS = SB_WARPS * 32, SB_STRIP4 = 32, SB_BLOCK_ROWS = 256, SB_DEPTH = 8;
constexpr int SB_MIN_ROWS = 64;     // a chunk has at least this many rows (bounds the number of partial sums)

template <int BT>
constexpr int sb_smem_bytes()
{
    // ring [SB_DEPTH][threads] float4, then delta [BT/4][SB_BLOCK_ROWS] float4; the reduction
    // ([warps][32 lanes][4 samples] float4 = 16 KiB) reuses the ring
    return SB_DEPTH * SB_THREADS * 16 + (BT / 4) * SB_BLOCK_ROWS * 16;
}

__device__ __forceinline__ void sb_cp_async16(unsigned dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void sb_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N_PENDING>
__device__ __forceinline__ void sb_cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N_PENDING) : "memory"); }

template <int BT>
__global__ void __launch_bounds__(SB_THREADS, BT <= 4 ? 4 : BT <= 8 ? 3 : 2)
k_delta_small_batch(const float* __restrict__ w_up, const float* __restrict__ delta_up, const float* __restrict__ a_l,
                    float* __restrict__ delta_l, float* __restrict__ partial, unsigned* __restrict__ counters,
                    int n_up, int n_l, int B, int rows_per_chunk, int chunks, int act)
{
    extern __shared__ __align__(16) unsigned char sb_smem[];
    float4* ring = reinterpret_cast<float4*>(sb_smem);                                   // [SB_DEPTH][threads]
    float4* d_sm = reinterpret_cast<float4*>(sb_smem + SB_DEPTH * SB_THREADS * 16);      // [BT/4][SB_BLOCK_ROWS]
    __shared__ bool is_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int strip = blockIdx.x, chunk = blockIdx.y;
    const int n4 = n_l >> 2;
    const int c4 = strip * SB_STRIP4 + lane;
    const bool col_ok = c4 < n4;
    const int row0 = chunk * rows_per_chunk;
    const int rows = min(rows_per_chunk, n_up - row0);
    const int my_rows = rows > warp ? (rows - warp + SB_WARPS - 1) / SB_WARPS : 0;     // rows warp, warp + 8, ...
    const float4* wp = reinterpret_cast<const float4*>(w_up) + (size_t)(row0 + warp) * n4 + (col_ok ? c4 : 0);
    const unsigned ring_u32 = (unsigned)__cvta_generic_to_shared(ring + tid);

    // prologue: my first SB_DEPTH - 1 rows are on their way (one group per row, empty past the end)
#pragma unroll
    for (int i = 0; i < SB_DEPTH - 1; ++i) {
        if (col_ok && i < my_rows) sb_cp_async16(ring_u32 + i * SB_THREADS * 16, wp + (size_t)i * SB_WARPS * n4);
        sb_cp_commit();
    }

    // running sums as pairs of samples, acc[p][c] = (sample 2p, sample 2p + 1) of column c: the two
    // multiply-adds of a pair are one packed instruction (fma.rn.f32x2; each half an ordinary fp32 fma)
    float2 acc[BT / 2][4];
#pragma unroll
    for (int p = 0; p < BT / 2; ++p)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[p][c] = make_float2(0.f, 0.f);

    int i = 0;     // index of my next row
    for (int blk0 = 0; blk0 < rows; blk0 += SB_BLOCK_ROWS) {
        const int blk_rows = min(SB_BLOCK_ROWS, rows - blk0);
        __syncthreads();      // the previous block's delta values are no longer read
        for (int idx = tid; idx < (BT / 4) * SB_BLOCK_ROWS; idx += SB_THREADS) {
            const int j = idx & (SB_BLOCK_ROWS - 1), b4 = idx / SB_BLOCK_ROWS;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (j < blk_rows) {
                const float* src = delta_up + (size_t)(4 * b4) * n_up + row0 + blk0 + j;
                if (4 * b4 + 0 < B) v.x = __ldcg(src);
                if (4 * b4 + 1 < B) v.y = __ldcg(src + n_up);
                if (4 * b4 + 2 < B) v.z = __ldcg(src + 2 * (size_t)n_up);
                if (4 * b4 + 3 < B) v.w = __ldcg(src + 3 * (size_t)n_up);
            }
            d_sm[idx] = v;
        }
        __syncthreads();
        const int i_end = min(my_rows, (blk0 + blk_rows - warp + SB_WARPS - 1) / SB_WARPS);   // my rows below the block's end
        for (; i < i_end; ++i) {
            const int nx = i + SB_DEPTH - 1;
            if (col_ok && nx < my_rows)
                sb_cp_async16(ring_u32 + (nx % SB_DEPTH) * SB_THREADS * 16, wp + (size_t)nx * SB_WARPS * n4);
            sb_cp_commit();
            sb_cp_wait<SB_DEPTH - 1>();      // the group of row i has landed
            const float4 wv = ring[(i % SB_DEPTH) * SB_THREADS + tid];
            const int j = warp + i * SB_WARPS - blk0;
            const float2 w2[4] = {make_float2(wv.x, wv.x), make_float2(wv.y, wv.y), make_float2(wv.z, wv.z), make_float2(wv.w, wv.w)};
#pragma unroll
            for (int b4 = 0; b4 < BT / 4; ++b4) {
                const float4 d = d_sm[b4 * SB_BLOCK_ROWS + j];
                const float2 d01 = make_float2(d.x, d.y), d23 = make_float2(d.z, d.w);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    acc[2 * b4][c] = __ffma2_rn(w2[c], d01, acc[2 * b4][c]);
                    acc[2 * b4 + 1][c] = __ffma2_rn(w2[c], d23, acc[2 * b4 + 1][c]);
                }
            }
        }
    }
    sb_cp_wait<0>();
    __syncthreads();      // the ring is free: the eight warps' sums meet there, four samples per round
    float4* red = ring;                                          // [8 warps][32 lanes][4 samples]
#pragma unroll
    for (int r = 0; r < BT / 4; ++r) {
#pragma unroll
        for (int sidx = 0; sidx < 4; ++sidx) {
            const float2* ap = acc[2 * r + (sidx >> 1)];      // the pair that holds sample 4r + sidx
            const float4 v = (sidx & 1) ? make_float4(ap[0].y, ap[1].y, ap[2].y, ap[3].y) : make_float4(ap[0].x, ap[1].x, ap[2].x, ap[3].x);
            red[(warp * 32 + lane) * 4 + sidx] = col_ok ? v : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        __syncthreads();
        if (tid < 128) {
            const int l = tid & 31, sidx = tid >> 5, b = 4 * r + sidx, c = strip * SB_STRIP4 + l;
            float4 sum = red[l * 4 + sidx];
#pragma unroll
            for (int q = 1; q < SB_WARPS; ++q) {
                const float4 t = red[(q * 32 + l) * 4 + sidx];
                sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
            }
            if (b < B && c < n4) reinterpret_cast<float4*>(partial)[((size_t)chunk * B + b) * n4 + c] = sum;
        }
        __syncthreads();
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(&counters[strip], 1u) == (unsigned)chunks - 1u;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // last CTA of the strip: every (sample, four columns) of the strip, chunks added in order
    for (int idx = tid; idx < B * SB_STRIP4; idx += SB_THREADS) {
        const int b = idx >> 5, c = strip * SB_STRIP4 + (idx & 31);
        if (c >= n4) continue;
        const float4* src = reinterpret_cast<const float4*>(partial) + (size_t)b * n4 + c;
        const size_t step = (size_t)B * n4;
        float4 sum = __ldcg(src);
#pragma unroll 8
        for (int q = 1; q < chunks; ++q) {
            const float4 t = __ldcg(src + q * step);
            sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
        }
        const float4 av = reinterpret_cast<const float4*>(a_l)[(size_t)b * n4 + c];
        reinterpret_cast<float4*>(delta_l)[(size_t)b * n4 + c] =
            make_float4(sum.x * lf_act_prime(av.x, act), sum.y * lf_act_prime(av.y, act),
                        sum.z * lf_act_prime(av.z, act), sum.w * lf_act_prime(av.w, act));
    }
    if (tid == 0) counters[strip] = 0u;   // ready for the next launch
}

// CTAs of the kernel (BT running sums per column) that one SM holds; asked of the runtime once.
template <int BT>
int sb_ctas_per_sm()
{
    static int per_device[64] = {};     // the attribute below belongs to a device's copy of the kernel
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    if (per_device[dev]) return per_device[dev];
    cudaFuncSetAttribute(k_delta_small_batch<BT>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb_smem_bytes<BT>());
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_delta_small_batch<BT>, SB_THREADS, sb_smem_bytes<BT>()) != cudaSuccess || n < 1)
        n = 1;
    per_device[dev] = n;
    return n;
}

// rows of w^{l+1} per chunk: as many chunks as fill the resident CTA slots once, none shorter than
// SB_MIN_ROWS rows
int sb_rows_per_chunk(int n_up, int n_l, int B)
{
    const int strips = ((n_l >> 2) + SB_STRIP4 - 1) / SB_STRIP4;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int per_sm = B <= 4 ? sb_ctas_per_sm<4>() : B <= 8 ? sb_ctas_per_sm<8>() : sb_ctas_per_sm<16>();
    int chunks = sms * per_sm / strips;
    const int most = (n_up + SB_MIN_ROWS - 1) / SB_MIN_ROWS;
    if (chunks > most) chunks = most;
    if (chunks < 1) chunks = 1;
    int rows = (n_up + chunks - 1) / chunks;
    rows = (rows + 7) & ~7;
    return rows;
}

}  // namespace

cudaError_t lfk_delta_gemm(const float* w_up, const float* delta_up, const float* a_l,
                           float* delta_l, int n_up, int n_l, int B, int act, cudaStream_t s)
{
    // M = B, Nn = n_l (neuron k of layer l), K = n_up (neuron j of layer l+1); w_up[j][k] is n-contiguous
    k_gemm_simt<true, false, EPI_DELTA><<<gemm_grid(B, n_l), 256, 0, s>>>(
        delta_up, w_up, delta_l, nullptr, a_l, B, n_l, n_up, n_up, n_l, n_l, 0.f, act);
    return cudaGetLastError();
}

namespace {

// ---- Eq. bp4 for a handful of samples (B <= 16) --------------------------------------------------
// gw[j][k] = sum_b delta[b][j] a[b][k] is then a store stream like the rank-1 writer of B = 1: 4B
// multiply-adds per 16 bytes stored, nothing to tile.  A thread keeps four columns of a (BT float4)
// in registers and walks the rows of its block; the block's delta values sit in shared memory as
// float4 over four samples (broadcast loads).  grid = 1024-column blocks x row chunks.
constexpr int GS_THREADS = 256, GS_ROWS = 32;

template <int BT>
__global__ void __launch_bounds__(GS_THREADS)
k_gw_small_batch(const float* __restrict__ delta_l, const float* __restrict__ a_prev, float* __restrict__ gw_l,
                 int n_out, int n_in, int B, const lf_sgd sgd)
{
    __shared__ __align__(16) float4 d_sm[(BT / 4) * GS_ROWS];     // [sample group][row of the chunk]
    const int n4 = n_in >> 2;
    const int c4 = blockIdx.x * GS_THREADS + threadIdx.x;
    const int row0 = blockIdx.y * GS_ROWS;
    const int rows = min(GS_ROWS, n_out - row0);
    for (int idx = threadIdx.x; idx < (BT / 4) * GS_ROWS; idx += GS_THREADS) {
        const int j = idx % GS_ROWS, b4 = idx / GS_ROWS;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < rows) {
            const float* src = delta_l + (size_t)(4 * b4) * n_out + row0 + j;
            if (4 * b4 + 0 < B) v.x = src[0];
            if (4 * b4 + 1 < B) v.y = src[n_out];
            if (4 * b4 + 2 < B) v.z = src[2 * (size_t)n_out];
            if (4 * b4 + 3 < B) v.w = src[3 * (size_t)n_out];
        }
        d_sm[idx] = v;
    }
    __syncthreads();
    if (c4 >= n4) return;
    float4 av[BT];
#pragma unroll
    for (int b = 0; b < BT; ++b)
        av[b] = b < B ? reinterpret_cast<const float4*>(a_prev)[(size_t)b * n4 + c4] : make_float4(0.f, 0.f, 0.f, 0.f);
    float4* out = reinterpret_cast<float4*>(gw_l) + (size_t)row0 * n4 + c4;
    const float4* wsub = sgd.w_sub ? reinterpret_cast<const float4*>(sgd.w_sub) + (size_t)row0 * n4 + c4 : nullptr;
#pragma unroll 2
    for (int j = 0; j < rows; ++j) {
        // two columns per packed multiply-add (fma.rn.f32x2: each half an ordinary fp32 fma, samples in order)
        float2 g01 = make_float2(0.f, 0.f), g23 = make_float2(0.f, 0.f);
#pragma unroll
        for (int b4 = 0; b4 < BT / 4; ++b4) {
            const float4 d = d_sm[b4 * GS_ROWS + j];
            const float dv[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 dd = make_float2(dv[q], dv[q]);
                const float4& ab = av[4 * b4 + q];
                g01 = __ffma2_rn(dd, make_float2(ab.x, ab.y), g01);
                g23 = __ffma2_rn(dd, make_float2(ab.z, ab.w), g23);
            }
        }
        float4 g = make_float4(g01.x, g01.y, g23.x, g23.y);
        if (wsub)   // fused update: w - eta * g, the weights streamed through once
            g = lf_sgd_apply4(sgd.eta, __ldcs(wsub + (size_t)j * n4), g);
        __stcs(out + (size_t)j * n4, g);
    }
}

}  // namespace

cudaError_t lfk_gw_gemm_fp32(const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                             int B, lf_sgd sgd, cudaStream_t s)
{
    if (B <= 16) {      // a handful of samples: a store stream, not a contraction
        dim3 grid(((n_in >> 2) + GS_THREADS - 1) / GS_THREADS, (n_out + GS_ROWS - 1) / GS_ROWS);
        if (B <= 4) k_gw_small_batch<4><<<grid, GS_THREADS, 0, s>>>(delta_l, a_prev, gw_l, n_out, n_in, B, sgd);
        else if (B <= 8) k_gw_small_batch<8><<<grid, GS_THREADS, 0, s>>>(delta_l, a_prev, gw_l, n_out, n_in, B, sgd);
        else k_gw_small_batch<16><<<grid, GS_THREADS, 0, s>>>(delta_l, a_prev, gw_l, n_out, n_in, B, sgd);
        return cudaGetLastError();
    }
    // M = n_out (j), Nn = n_in (k), K = B; both operands are contiguous along their M / N index
    k_gemm_simt<false, false, EPI_PLAIN><<<gemm_grid(n_out, n_in), 256, 0, s>>>(
        delta_l, a_prev, gw_l, nullptr, sgd.w_sub, n_out, n_in, B, n_out, n_in, n_in, sgd.eta, LF_ACT_SIGMOID);
    return cudaGetLastError();
}

cudaError_t lfk_grad_b_colsum(const float* delta_l, float* gb_l, int N, int B, cudaStream_t s)
{
    k_grad_b_colsum<<<(N + 31) / 32, 256, 0, s>>>(delta_l, gb_l, N, B);
    return cudaGetLastError();
}

// ---- Eq. bp2 for B <= 16 samples: scratch sizes and launch ------------------------------------------
int lfk_small_batch_max() { return 16; }

size_t lfk_delta_small_batch_scratch_floats(int n_up, int n_l, int B)
{
    const int rows = sb_rows_per_chunk(n_up, n_l, B);
    const int chunks = (n_up + rows - 1) / rows;
    return (size_t)chunks * B * n_l;
}

cudaError_t lfk_delta_small_batch(const float* w_up, const float* delta_up, const float* a_l, float* delta_l,
                                  float* partial, unsigned* counters, int n_up, int n_l, int B, int act, cudaStream_t s)
{
    const int rows = sb_rows_per_chunk(n_up, n_l, B);
    const int chunks = (n_up + rows - 1) / rows;
    const int strips = ((n_l >> 2) + SB_STRIP4 - 1) / SB_STRIP4;
    dim3 grid(strips, chunks);
    if (B <= 4)
        k_delta_small_batch<4><<<grid, SB_THREADS, sb_smem_bytes<4>(), s>>>(w_up, delta_up, a_l, delta_l, partial, counters, n_up, n_l, B, rows, chunks, act);
    else if (B <= 8)
        k_delta_small_batch<8><<<grid, SB_THREADS, sb_smem_bytes<8>(), s>>>(w_up, delta_up, a_l, delta_l, partial, counters, n_up, n_l, B, rows, chunks, act);
    else
        k_delta_small_batch<16><<<grid, SB_THREADS, sb_smem_bytes<16>(), s>>>(w_up, delta_up, a_l, delta_l, partial, counters, n_up, n_l, B, rows, chunks, act);
    return cudaGetLastError();
}
