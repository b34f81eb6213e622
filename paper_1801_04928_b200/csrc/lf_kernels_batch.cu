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

cudaError_t lfk_delta_gemm(const float* w_up, const float* delta_up, const float* a_l,
                           float* delta_l, int n_up, int n_l, int B, int act, cudaStream_t s)
{
    // M = B, Nn = n_l (neuron k of layer l), K = n_up (neuron j of layer l+1); w_up[j][k] is n-contiguous
    k_gemm_simt<true, false, EPI_DELTA><<<gemm_grid(B, n_l), 256, 0, s>>>(
        delta_up, w_up, delta_l, nullptr, a_l, B, n_l, n_up, n_up, n_l, n_l, 0.f, act);
    return cudaGetLastError();
}

cudaError_t lfk_gw_gemm_fp32(const float* delta_l, const float* a_prev, float* gw_l, int n_out, int n_in,
                             int B, lf_sgd sgd, cudaStream_t s)
{
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
