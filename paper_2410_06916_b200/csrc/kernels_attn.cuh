// GQA decode attention over the paged KV cache for the <= 16 new rows of one forward chunk, with
// the causal mask across those rows.  Split-KV: each CTA owns one (query head, 256-position chunk);
// chunks are anchored at multiples of 256 positions and combined in chunk order, so a row's result
// does not depend on how many other rows are in flight.
#pragma once
#include "common.cuh"
#include "kernels_gemm_tc.cuh"

namespace swk {

constexpr int ATTN_THREADS = 128;

// grid = (H, max_splits), block = 128.  One CTA = one query head x one chunk of ATTN_CHUNK positions.
// The chunk's K and V rows are contiguous per page in the pool, so they are brought into shared memory
// with a handful of bulk copies (one per page and per K/V) signalled on an mbarrier; the arithmetic then
// runs entirely out of shared memory:
//   scores : thread (j, half) takes position j and one half of the head dimension for all rows; its
//            16-byte reads of K and q start at a chunk index rotated by j, which spreads the 128-byte-
//            strided rows over all banks;
//   softmax: one warp per row;
//   output : thread d accumulates sum_j p[r][j] * V[j][d] for all rows.
// Dynamic smem: 2 * ATTN_CHUNK * dh * sizeof(T) (K, V) + MR*dh*4 (q) + 3*MR*ATTN_CHUNK*4 (score halves, p).
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

    extern __shared__ __align__(128) unsigned char attn_smem[];
    T* Ks = reinterpret_cast<T*>(attn_smem);               // [ATTN_CHUNK][dh]
    T* Vs = Ks + ATTN_CHUNK * dh;                          // [ATTN_CHUNK][dh]
    float* qs = reinterpret_cast<float*>(Vs + ATTN_CHUNK * dh);   // [MR][dh], pre-scaled
    float* sc = qs + MR * dh;                              // [2][MR][ATTN_CHUNK] partial scores of the two halves
    float* ps = sc + 2 * MR * ATTN_CHUNK;                  // [MR][ATTN_CHUNK] probabilities
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ float row_m[MR], row_l[MR];
    __shared__ int load_ok;
    const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&bar_storage);

    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // one bulk copy per page piece of K and of V
        const int piece = min(L.page_size, ATTN_CHUNK);                 // positions per piece (both powers of two)
        const int n_pieces = (len + piece - 1) / piece;
        const uint32_t piece_bytes = (uint32_t)(piece * dh * sizeof(T));
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2u * n_pieces * piece_bytes) : "memory");
        for (int i = 0; i < n_pieces; ++i) {
            const int pos = c0 + i * piece;
            const int page = page_table[pos >> L.page_shift], slot = pos & (L.page_size - 1);
            const T* ksrc = kv_pool + L.offset(page, block, 0, kvh, slot);
            const T* vsrc = kv_pool + L.offset(page, block, 1, kvh, slot);
            const uint32_t kdst = (uint32_t)__cvta_generic_to_shared(Ks + (size_t)i * piece * dh);
            const uint32_t vdst = (uint32_t)__cvta_generic_to_shared(Vs + (size_t)i * piece * dh);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(kdst), "l"(ksrc), "r"(piece_bytes), "r"(bar) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(vdst), "l"(vsrc), "r"(piece_bytes), "r"(bar) : "memory");
        }
    }
    for (int i = tid; i < MR * dh; i += ATTN_THREADS) {
        const int r = i / dh, d = i - r * dh;
        qs[i] = r < n_rows ? q[((size_t)r * n_heads + h) * dh + d] * scale : 0.f;
    }
    __syncthreads();                                       // barrier initialised, q staged
    if (tid == 0) {                                        // bounded wait for the copies, result shared with the block
        const long long t0 = clock64();
        int ok = 0;
        for (uint32_t it = 0; !ok; ++it) {
            uint32_t done;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(done) : "r"(bar) : "memory");
            if (done) ok = 1;
            else if ((it & 63u) == 63u && clock64() - t0 > 3000000000LL) break;
        }
        load_ok = ok;
    }
    __syncthreads();
    if (!load_ok) {
        if (tid == 0) const_cast<DevState*>(st)->error = 3;
        return;
    }

    // phase 1: partial scores
    {
        const int half_d = dh >> 1;
        const int chunks = half_d / VEC > 0 ? half_d / VEC : 1;          // 16-byte chunks per half row
        const int j = tid & (ATTN_CHUNK - 1), hh = tid >> 6;
        if (j < len && hh < 2) {
            float acc[MR];
#pragma unroll
            for (int r = 0; r < MR; ++r) acc[r] = 0.f;
            const T* krow = Ks + (size_t)j * dh + hh * half_d;
            const float* qrow = qs + hh * half_d;
            for (int c = 0; c < chunks; ++c) {
                const int cc = ((c + j) & (chunks - 1)) * VEC;      // chunks is a power of two
                float kv[VEC];
                load_vec(krow + cc, kv);
#pragma unroll
                for (int r = 0; r < MR; ++r) {
#pragma unroll
                    for (int e = 0; e < VEC; e += 4) {
                        const float4 qq = *reinterpret_cast<const float4*>(qrow + r * dh + cc + e);
                        acc[r] = fmaf(kv[e], qq.x, acc[r]);
                        acc[r] = fmaf(kv[e + 1], qq.y, acc[r]);
                        acc[r] = fmaf(kv[e + 2], qq.z, acc[r]);
                        acc[r] = fmaf(kv[e + 3], qq.w, acc[r]);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < MR; ++r) sc[(hh * MR + r) * ATTN_CHUNK + j] = acc[r];
        }
    }
    __syncthreads();

    // phase 2: per-row max, exponentials, sum (one warp per row, rows strided over the warps)
    const int lane = tid & 31, warp = tid >> 5;
    for (int r = warp; r < n_rows; r += ATTN_THREADS / 32) {
        float m = -INFINITY;
        for (int j = lane; j < len; j += 32) {
            const float v = (c0 + j <= pos0 + r) ? sc[r * ATTN_CHUNK + j] + sc[(MR + r) * ATTN_CHUNK + j] : -INFINITY;
            ps[r * ATTN_CHUNK + j] = v;
            m = fmaxf(m, v);
        }
        m = warp_max(m);
        float l = 0.f;
        for (int j = lane; j < len; j += 32) {
            const float p = (m == -INFINITY) ? 0.f : expf(ps[r * ATTN_CHUNK + j] - m);
            ps[r * ATTN_CHUNK + j] = p;
            l += p;
        }
        l = warp_sum(l);
        if (lane == 0) { row_m[r] = m; row_l[r] = l; }
    }
    __syncthreads();

    // phase 3: out[r][d] = sum_j p[r][j] * V[j][d]; one thread per d, positions taken four at a time so that
    // one 16-byte read of p feeds four multiply-adds (same summation order as one at a time)
    const int len4 = len & ~3;
    for (int d = tid; d < dh; d += ATTN_THREADS) {
        float acc[MR];
#pragma unroll
        for (int r = 0; r < MR; ++r) acc[r] = 0.f;
        for (int j = 0; j < len4; j += 4) {
            const float v0 = to_float(Vs[(size_t)j * dh + d]), v1 = to_float(Vs[(size_t)(j + 1) * dh + d]);
            const float v2 = to_float(Vs[(size_t)(j + 2) * dh + d]), v3 = to_float(Vs[(size_t)(j + 3) * dh + d]);
#pragma unroll
            for (int r = 0; r < MR; ++r) {
                const float4 p4 = *reinterpret_cast<const float4*>(ps + r * ATTN_CHUNK + j);
                acc[r] = fmaf(p4.x, v0, acc[r]);
                acc[r] = fmaf(p4.y, v1, acc[r]);
                acc[r] = fmaf(p4.z, v2, acc[r]);
                acc[r] = fmaf(p4.w, v3, acc[r]);
            }
        }
        for (int j = len4; j < len; ++j) {
            const float v = to_float(Vs[(size_t)j * dh + d]);
#pragma unroll
            for (int r = 0; r < MR; ++r) acc[r] = fmaf(ps[r * ATTN_CHUNK + j], v, acc[r]);
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
