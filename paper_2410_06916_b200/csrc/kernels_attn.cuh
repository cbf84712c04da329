// GQA decode attention over the paged KV cache for the <= 16 new rows of one forward chunk, with
// the causal mask across those rows.  Split-KV: each CTA owns one (query head, 256-position chunk);
// chunks are anchored at multiples of 256 positions and combined in chunk order, so a row's result
// does not depend on how many other rows are in flight.
#pragma once
#include "common.cuh"
#include "kernels_gemm_tc.cuh"

namespace swk {

constexpr int ATTN_THREADS = 128;

// grid = (H, max_splits).  Dynamic smem: MR*dh floats (q) + MR*ATTN_CHUNK floats (scores) + 2*MR.
// Writes unnormalised partial outputs o_part[h][s][r][dh] and (m, l) pairs ml_part[h][s][r].
template <typename T, int MR>
__global__ void __launch_bounds__(ATTN_THREADS)
attn_split_kernel(const DevState* st, const float* __restrict__ q, const T* __restrict__ kv_pool,
                  const int* __restrict__ page_table, KvLayout L, int block, int n_heads, int max_splits,
                  float scale, float* __restrict__ o_part, float2* __restrict__ ml_part)
{
    pdl_enter();
    constexpr int VEC = Vec<T>::N;
    const int n_rows = min(st->n_rows, MR);
    if (n_rows == 0) return;
    const int pos0 = st->pos0;
    const int total = pos0 + n_rows;                       // positions visible to the last row
    const int h = blockIdx.x, s = blockIdx.y;
    const int c0 = s * ATTN_CHUNK;
    if (c0 >= total) return;
    const int len = min(ATTN_CHUNK, total - c0);
    const int dh = L.head_dim;
    const int kvh = h / (n_heads / L.n_kv_heads);
    const int tid = threadIdx.x;

    extern __shared__ __align__(16) float smem_f[];
    float* qs = smem_f;                                    // [MR][dh], pre-scaled
    float* sc = qs + MR * dh;                              // [MR][ATTN_CHUNK]
    float* row_m = sc + MR * ATTN_CHUNK;                   // [MR]
    float* row_l = row_m + MR;                             // [MR]

    for (int i = tid; i < MR * dh; i += ATTN_THREADS) {
        const int r = i / dh, d = i - r * dh;
        qs[i] = r < n_rows ? q[((size_t)r * n_heads + h) * dh + d] * scale : 0.f;
    }
    __syncthreads();

    // phase 1: scores.  One thread per position; K row read in 16-byte pieces.
    for (int j = tid; j < len; j += ATTN_THREADS) {
        const int pos = c0 + j;
        const T* kp = kv_pool + L.offset(page_table[pos >> L.page_shift], block, 0, kvh, pos & (L.page_size - 1));
        float acc[MR];
#pragma unroll
        for (int r = 0; r < MR; ++r) acc[r] = 0.f;
        for (int d = 0; d < dh; d += VEC) {
            float kv[VEC];
            load_vec(kp + d, kv);
#pragma unroll
            for (int r = 0; r < MR; ++r) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[r] = fmaf(kv[e], qs[r * dh + d + e], acc[r]);
            }
        }
#pragma unroll
        for (int r = 0; r < MR; ++r) sc[r * ATTN_CHUNK + j] = (pos <= pos0 + r) ? acc[r] : -INFINITY;
    }
    __syncthreads();

    // phase 2: per-row max, exponentials, sum (one warp per row, rows strided over the warps)
    const int lane = tid & 31, warp = tid >> 5;
    for (int r = warp; r < n_rows; r += ATTN_THREADS / 32) {
        float m = -INFINITY;
        for (int j = lane; j < len; j += 32) m = fmaxf(m, sc[r * ATTN_CHUNK + j]);
        m = warp_max(m);
        float l = 0.f;
        for (int j = lane; j < len; j += 32) {
            const float p = (m == -INFINITY) ? 0.f : expf(sc[r * ATTN_CHUNK + j] - m);
            sc[r * ATTN_CHUNK + j] = p;
            l += p;
        }
        l = warp_sum(l);
        if (lane == 0) { row_m[r] = m; row_l[r] = l; }
    }
    __syncthreads();

    // phase 3: out[r][d] = sum_j p[r][j] * V[j][d]; one thread per d
    for (int d = tid; d < dh; d += ATTN_THREADS) {
        float acc[MR];
#pragma unroll
        for (int r = 0; r < MR; ++r) acc[r] = 0.f;
        for (int j = 0; j < len; ++j) {
            const int pos = c0 + j;
            const T* vp = kv_pool + L.offset(page_table[pos >> L.page_shift], block, 1, kvh, pos & (L.page_size - 1));
            const float v = to_float(vp[d]);
#pragma unroll
            for (int r = 0; r < MR; ++r) acc[r] = fmaf(sc[r * ATTN_CHUNK + j], v, acc[r]);
        }
#pragma unroll
        for (int r = 0; r < MR; ++r)
            if (r < n_rows) o_part[(((size_t)h * max_splits + s) * ROWS + r) * dh + d] = acc[r];
    }
    if (tid < n_rows) ml_part[((size_t)h * max_splits + s) * ROWS + tid] = make_float2(row_m[tid], row_l[tid]);
}

// grid = (H, rows), block = dh threads.  Combines the splits in chunk order.
__global__ void attn_combine_kernel(const DevState* st, const float* __restrict__ o_part,
                                    const float2* __restrict__ ml_part, int max_splits, int n_heads, int dh,
                                    float* __restrict__ out, __nv_bfloat16* __restrict__ planes)
{
    pdl_enter();
    const int r = blockIdx.y;
    if (r >= st->n_rows) return;
    const int h = blockIdx.x, d = threadIdx.x;
    const int total = st->pos0 + st->n_rows;
    const int n_splits = (total + ATTN_CHUNK - 1) / ATTN_CHUNK;
    float M = -INFINITY;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, ml_part[((size_t)h * max_splits + s) * ROWS + r].x);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float2 ml = ml_part[((size_t)h * max_splits + s) * ROWS + r];
        const float w = (ml.x == -INFINITY) ? 0.f : expf(ml.x - M);
        num += w * o_part[(((size_t)h * max_splits + s) * ROWS + r) * dh + d];
        den += w * ml.y;
    }
    const float v = num / den;
    out[((size_t)r * n_heads + h) * dh + d] = v;
    if (planes) store_hi_lo(planes, r, n_heads * dh, h * dh + d, v);
}

} // namespace swk
