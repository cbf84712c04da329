// Skinny weight-streaming GEMM, SIMT form:  Ypart[s][r][n] = sum_{k in split s} X[r][k] * W[n][k]
// for at most 16 rows r.  Used for fp32 models and as the reference the tensor-core path is tested
// against.  Each output element is reduced in an order that does not depend on the row count, so a
// row computed alone (drafting, vanilla decoding) and the same row inside a verification batch give
// identical bits.
#pragma once
#include "common.cuh"

namespace swk {

constexpr int GEMM_SIMT_THREADS = 256;
constexpr int GEMM_SIMT_R = 4;                                   // weight rows per warp
constexpr int GEMM_SIMT_TILE_N = (GEMM_SIMT_THREADS / 32) * GEMM_SIMT_R;

// Activations X are fp32 (nothing but the weights and the KV cache is ever rounded to bf16); weights
// are T.  grid = (ceil(N / 32), n_split); dynamic smem = MR * Kc * 4 bytes.
// Kc is a multiple of 32 * VEC; K a multiple of VEC; X rows are ldx elements apart (16-byte aligned).
template <typename T, int MR>
__global__ void __launch_bounds__(GEMM_SIMT_THREADS)
gemm_simt_kernel(const DevState* st, const float* __restrict__ X, int ldx, const T* __restrict__ W,
                 float* __restrict__ Ypart, int N, int K, int Kc)
{
    pdl_enter();
    constexpr int VEC = Vec<T>::N;
    constexpr int R = GEMM_SIMT_R;
    const int n_rows = min(st->n_rows, MR);
    if (n_rows == 0) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);              // [MR][Kc]

    const int k0 = blockIdx.y * Kc;
    const int klen = min(Kc, K - k0);
    if (klen <= 0) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // stage the X rows of this K range (rows beyond n_rows are zero)
    for (int m = 0; m < MR; ++m) {
        for (int kk = tid * 4; kk < klen; kk += GEMM_SIMT_THREADS * 4) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m < n_rows) v = *reinterpret_cast<const float4*>(X + (size_t)m * ldx + k0 + kk);
            *reinterpret_cast<float4*>(xs + (size_t)m * Kc + kk) = v;
        }
    }
    __syncthreads();

    const int n_base = (blockIdx.x * (GEMM_SIMT_THREADS / 32) + warp) * R;
    if (n_base >= N) return;
    float acc[R][MR];
#pragma unroll
    for (int rr = 0; rr < R; ++rr)
#pragma unroll
        for (int m = 0; m < MR; ++m) acc[rr][m] = 0.f;

    const T* wrow[R];
#pragma unroll
    for (int rr = 0; rr < R; ++rr) wrow[rr] = W + (size_t)min(n_base + rr, N - 1) * K + k0;

#pragma unroll 2
    for (int kk = lane * VEC; kk < klen; kk += 32 * VEC) {
        float w[R][VEC];
#pragma unroll
        for (int rr = 0; rr < R; ++rr) load_vec_stream(wrow[rr] + kk, w[rr]);
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            float x[VEC];
#pragma unroll
            for (int e = 0; e < VEC; e += 4) {
                const float4 v = *reinterpret_cast<const float4*>(xs + (size_t)m * Kc + kk + e);
                x[e] = v.x; x[e + 1] = v.y; x[e + 2] = v.z; x[e + 3] = v.w;
            }
#pragma unroll
            for (int rr = 0; rr < R; ++rr)
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[rr][m] = fmaf(w[rr][e], x[e], acc[rr][m]);
        }
    }

    float* out = Ypart + (size_t)blockIdx.y * ROWS * N;
#pragma unroll
    for (int rr = 0; rr < R; ++rr)
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            const float v = warp_sum(acc[rr][m]);
            if (lane == 0 && m < n_rows && n_base + rr < N) out[(size_t)m * N + n_base + rr] = v;
        }
}

} // namespace swk
