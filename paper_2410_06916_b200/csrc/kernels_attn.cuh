// GQA decode attention over the paged KV cache for the <= 16 new rows of one forward chunk, with
// the causal mask across those rows.  Split-KV: each CTA owns one (query head, 64-position chunk);
// chunks are anchored at multiples of 64 positions and merged in chunk order, so a row's result
// does not depend on how many other rows are in flight.  Two split kernels: attn_stream_kernel
// (head_dim 128: K and V go straight from the cache into registers) and attn_split_kernel (any
// head size, K and V staged in shared memory); the merge is attn_combine_kernel, or the tail of
// attn_stream_kernel itself for one-row forwards.
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
            const int pj = c0 + j;                          // cached context, or a row of the forward this row may see
            const bool vis = pj < pos0 || ((st->row_vis[r] >> (pj - pos0)) & 1u) != 0u;
            const float v = vis ? sc[r * ATTN_CHUNK + j] + sc[(MR + r) * ATTN_CHUNK + j] : -INFINITY;
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

// Merges the splits of one (head, row) in chunk order; called by all blockDim.x = dh threads of a block.
// comb_sh: 2 * max_splits floats, wmax_sh: 32 floats of shared memory.  The (m, l) pairs are fetched once per
// block, spread over the threads, and the partial outputs are read eight splits at a time with independent
// loads, so this costs a few trips to L2 rather than one per split; the sums themselves run over the splits
// in ascending order.
__device__ __forceinline__ void combine_row(int pos0, int r, int h, const float* __restrict__ o_part,
                                            const float2* __restrict__ ml_part, int max_splits, int n_heads, int dh,
                                            float* __restrict__ out, __nv_bfloat16* __restrict__ planes,
                                            float* comb_sh, float* wmax_sh, int part_rows = ROWS, int row_shift = 0)
{
    // row_shift: where row r of this sequence sits in the partial-result and output buffers (a sequence inside a larger chunk)
    const int d = threadIdx.x;
    // row r sees positions <= pos0 + r: later splits hold nothing for it (and, when the rows were processed in
    // groups, were not written for it at all)
    const int n_splits = (pos0 + r + 1 + ATTN_CHUNK - 1) / ATTN_CHUNK;
    float* w_sh = comb_sh;                    // [n_splits] exp(m_s - M), 0 for empty splits
    float* l_sh = comb_sh + max_splits;       // [n_splits]
    const size_t base = (size_t)h * max_splits;

    // the first 16 splits' partial outputs are requested before anything else: they do not depend on the weights
    constexpr int CB = 16;
    const float* op = o_part + (base * part_rows + r + row_shift) * dh + d;
    const size_t stride = (size_t)part_rows * dh;
    float o[CB];
#pragma unroll
    for (int i = 0; i < CB; ++i) o[i] = i < n_splits ? __ldcg(op + (size_t)i * stride) : 0.f;

    float mx = -INFINITY;
    for (int s = d; s < n_splits; s += blockDim.x) {
        const float2 ml = __ldcg(ml_part + (base + s) * part_rows + r + row_shift);
        w_sh[s] = ml.x;
        l_sh[s] = ml.y;
        mx = fmaxf(mx, ml.x);
    }
    mx = warp_max(mx);
    if ((d & 31) == 0) wmax_sh[d >> 5] = mx;
    __syncthreads();
    float M = -INFINITY;
    for (int wi = 0; wi < (int)(blockDim.x + 31) / 32; ++wi) M = fmaxf(M, wmax_sh[wi]);
    for (int s = d; s < n_splits; s += blockDim.x) {
        const float m = w_sh[s];
        w_sh[s] = (m == -INFINITY) ? 0.f : expf(m - M);
    }
    __syncthreads();

    float num = 0.f, den = 0.f;
    for (int s0 = 0; s0 < n_splits; s0 += CB) {
        if (s0 > 0) {
#pragma unroll
            for (int i = 0; i < CB; ++i) o[i] = s0 + i < n_splits ? __ldcg(op + (size_t)(s0 + i) * stride) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < CB; ++i) {
            if (s0 + i < n_splits) {
                num = fmaf(w_sh[s0 + i], o[i], num);
                den = fmaf(w_sh[s0 + i], l_sh[s0 + i], den);
            }
        }
    }
    const float v = num / den;
    out[((size_t)(r + row_shift) * n_heads + h) * dh + d] = v;
    if (planes) store_hi_lo(planes, r + row_shift, n_heads * dh, h * dh + d, v);
}

// ---------------------------------------------------------------------------------------------
// Streaming form for head_dim == 128: no shared-memory staging of K and V; every byte of the cache is
// loaded once, straight into registers, by coalesced warp loads with many rows in flight per warp.
// grid = (H, max_splits, row groups), block = 128.  A CTA takes MR consecutive rows of the forward chunk
// (blockIdx.z picks the group).  Warp w owns positions [16w, 16w + 16) of the chunk and takes
// them in two batches of eight.  Within a batch, with lane = 8 * pg + dl:
//   K : lane holds elements {32c + 4dl .. +3, c = 0..3} of rows pg and pg + 4 (eight lanes per row),
//       so a score is a 16-term chain per lane followed by a three-level xor tree over dl.  The tree is
//       "packed": while a lane holds an even number of sums it keeps one half and hands the other to
//       its partner, which yields the same additions as the full butterfly at a fraction of the
//       shuffles and leaves every (row, position) score in one owner lane (times replication);
//   softmax: the owner lanes do the running max / exponentials / sums, trees over the position lanes;
//   V : lane holds elements [4 lane, 4 lane + 4) of all eight rows; probabilities and rescale factors
//       reach all lanes through a small per-warp shared array.
// Finally the four warps' partial results are merged in warp order.  A query row's arithmetic does not
// depend on MR or on how many other rows are present: masked positions enter with probability exactly
// 0 and a rescale factor of exactly 1 where nothing is visible yet.
// Same outputs as attn_split_kernel: o_part[h][s][r][dh] (unnormalised) and ml_part[h][s][r].
constexpr int ATTN_BATCH = 8;

template <typename T>
__device__ __forceinline__ float4 load_row4(const T* p);
template <>
__device__ __forceinline__ float4 load_row4<float>(const float* p)
{
    return __ldg(reinterpret_cast<const float4*>(p));
}
template <>
__device__ __forceinline__ float4 load_row4<__nv_bfloat16>(const __nv_bfloat16* p)
{
    const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
    float4 f;
    f.x = __uint_as_float(u.x << 16);
    f.y = __uint_as_float(u.x & 0xFFFF0000u);
    f.z = __uint_as_float(u.y << 16);
    f.w = __uint_as_float(u.y & 0xFFFF0000u);
    return f;
}

// One level of the xor tree over N per-lane sums.  Even N: the lane with `upper` clear keeps sums
// [0, N/2) and adds the partner's copies of them, the other lane keeps [N/2, N); N/2 sums remain, in
// v[0 .. N/2).  Odd N: plain butterfly, N sums remain.
template <int N>
__device__ __forceinline__ void fold_level(float* v, int off, bool upper)
{
    if constexpr (N % 2 == 0) {
        constexpr int H = N / 2;
#pragma unroll
        for (int i = 0; i < H; ++i) {
            const float keep = upper ? v[i + H] : v[i];
            const float send = upper ? v[i] : v[i + H];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) v[i] += __shfl_xor_sync(0xffffffffu, v[i], off);
    }
}
__host__ __device__ constexpr int folded(int n) { return n % 2 == 0 ? n / 2 : n; }

template <typename T, int MR>
__global__ void __launch_bounds__(ATTN_THREADS, MR == 1 ? 5 : (MR <= 12 ? 3 : 2))
attn_stream_kernel(const DevState* st, const float* __restrict__ q, const T* __restrict__ kv_pool,
                   const int* __restrict__ page_table, KvLayout L, int block, int n_heads, int max_splits,
                   float scale, float* __restrict__ o_part, float2* __restrict__ ml_part,
                   int* __restrict__ head_counters, float* __restrict__ out, __nv_bfloat16* __restrict__ planes)
{
    pdl_enter();
    constexpr int DH = 128, NW = ATTN_THREADS / 32, PER_WARP = ATTN_CHUNK / NW;
    static_assert(PER_WARP == 2 * ATTN_BATCH, "two batches per warp");
    constexpr int N1 = MR, N2 = folded(N1), N3 = folded(N2);       // sums per lane after each tree level
    // blockIdx.z selects a group of MR consecutive rows of the forward chunk; everything below is relative to it
    const int row0 = blockIdx.z * MR;
    const int n_rows = min(st->n_rows - row0, MR);
    if (n_rows <= 0) return;
    const int pos0 = st->pos0 + row0;                       // position of the group's first row
    const int total = pos0 + n_rows;                        // positions visible to the group's last row
    q += (size_t)row0 * n_heads * 128;
    const int h = blockIdx.x, s = blockIdx.y;
    const int c0 = s * ATTN_CHUNK;
    if (c0 >= total) return;
    const int len = min(ATTN_CHUNK, total - c0);
    const int kvh = h / (n_heads / L.n_kv_heads);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int pg = lane >> 3, dl = lane & 7;
    const bool b2 = (lane >> 2) & 1, b1 = (lane >> 1) & 1, b0 = lane & 1;
    // what this lane owns after the tree: position pi of the batch and rows [row_base, row_base + N3)
    const int pi = pg + (b2 ? 4 : 0);
    int row_base = 0;
    if (N1 % 2 == 0) row_base += b1 ? N2 : 0;
    if (N2 % 2 == 0) row_base += b0 ? N3 : 0;

    __shared__ float4 q_sh[MR][32];
    __shared__ __align__(16) float part_acc[NW][MR][DH];
    __shared__ float2 part_ml[NW][MR];
    __shared__ __align__(16) float p_sh[NW][MR][ATTN_BATCH];
    __shared__ float corr_sh[NW][MR];
    __shared__ unsigned vis_sh[ROWS];
    if (tid < ROWS) vis_sh[tid] = st->row_vis[tid];

    for (int i = tid; i < MR * 32; i += ATTN_THREADS) {
        const int r = i >> 5, c = i & 31;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < n_rows) {
            v = *reinterpret_cast<const float4*>(q + ((size_t)r * n_heads + h) * DH + c * 4);
            v.x *= scale; v.y *= scale; v.z *= scale; v.w *= scale;
        }
        q_sh[r][c] = v;
    }
    __syncthreads();

    float m_own[N3], l_own[N3];
#pragma unroll
    for (int t = 0; t < N3; ++t) { m_own[t] = -INFINITY; l_own[t] = 0.f; }
    float4 acc[MR];
#pragma unroll
    for (int r = 0; r < MR; ++r) acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);
    const size_t v_off = (size_t)L.n_kv_heads * L.page_size * DH;      // from a K row to the V row of the same slot

#pragma unroll 1
    for (int b = 0; b < 2; ++b) {
        const int j0 = w * PER_WARP + b * ATTN_BATCH;
        if (j0 >= len) break;
        // rows past the end re-read the last one (finite values); they are masked below
        float4 kx[2][4], vx[ATTN_BATCH];
#pragma unroll
        for (int sl = 0; sl < 2; ++sl) {
            const int pos = c0 + min(j0 + pg + 4 * sl, len - 1);
            const int page = __ldg(page_table + (pos >> L.page_shift));
            const T* kp = kv_pool + L.offset(page, block, 0, kvh, pos & (L.page_size - 1)) + dl * 4;
#pragma unroll
            for (int c = 0; c < 4; ++c) kx[sl][c] = load_row4<T>(kp + 32 * c);
        }
#pragma unroll
        for (int i = 0; i < ATTN_BATCH; ++i) {
            const int pos = c0 + min(j0 + i, len - 1);
            const int page = __ldg(page_table + (pos >> L.page_shift));
            vx[i] = load_row4<T>(kv_pool + L.offset(page, block, 0, kvh, pos & (L.page_size - 1)) + v_off + lane * 4);
        }

        // partial scores: sc[sl * MR + r] over this lane's 16 elements
        float sc[2 * MR];
#pragma unroll
        for (int r = 0; r < MR; ++r) {
            float s0 = 0.f, s1 = 0.f;
            if (r < n_rows) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float4 q4 = q_sh[r][8 * c + dl];
                    s0 = fmaf(kx[0][c].x, q4.x, s0); s0 = fmaf(kx[0][c].y, q4.y, s0);
                    s0 = fmaf(kx[0][c].z, q4.z, s0); s0 = fmaf(kx[0][c].w, q4.w, s0);
                    s1 = fmaf(kx[1][c].x, q4.x, s1); s1 = fmaf(kx[1][c].y, q4.y, s1);
                    s1 = fmaf(kx[1][c].z, q4.z, s1); s1 = fmaf(kx[1][c].w, q4.w, s1);
                }
            }
            sc[r] = s0; sc[MR + r] = s1;
        }
        fold_level<2 * MR>(sc, 4, b2);          // -> N1 = MR sums: all rows, position pi
        fold_level<N1>(sc, 2, b1);              // -> N2
        fold_level<N2>(sc, 1, b0);              // -> N3 sums: rows row_base .., position pi

        __syncwarp();                           // previous batch's readers of p_sh are done
#pragma unroll
        for (int t = 0; t < N3; ++t) {
            const int r = row_base + t;
            float x = sc[t];
            {                                                          // visibility among the forward's rows; also covers positions past the end
                const int dlt = c0 + j0 + pi - pos0 + row0;            // index among the forward's rows; negative = cached context
                if (dlt >= 0 && (dlt >= ROWS || ((vis_sh[min(row0 + r, ROWS - 1)] >> dlt) & 1u) == 0u)) x = -INFINITY;
            }
            float bm = x;
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
            const float mn = fmaxf(m_own[t], bm);
            float corr = 1.f, p = 0.f;
            if (mn != -INFINITY) {
                corr = (m_own[t] == -INFINITY) ? 0.f : expf(m_own[t] - mn);
                p = (x == -INFINITY) ? 0.f : expf(x - mn);
            }
            float ps = p;
            ps += __shfl_xor_sync(0xffffffffu, ps, 4);
            ps += __shfl_xor_sync(0xffffffffu, ps, 8);
            ps += __shfl_xor_sync(0xffffffffu, ps, 16);
            l_own[t] = fmaf(l_own[t], corr, ps);
            m_own[t] = mn;
            p_sh[w][r][pi] = p;
            if (pi == 0) corr_sh[w][r] = corr;
        }
        __syncwarp();

#pragma unroll
        for (int r = 0; r < MR; ++r) {
            if (r < n_rows) {
                const float corr = corr_sh[w][r];
                const float4 pa = *reinterpret_cast<const float4*>(&p_sh[w][r][0]);
                const float4 pb = *reinterpret_cast<const float4*>(&p_sh[w][r][4]);
                const float pp[ATTN_BATCH] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
                float4 a = acc[r];
                a.x *= corr; a.y *= corr; a.z *= corr; a.w *= corr;
#pragma unroll
                for (int i = 0; i < ATTN_BATCH; ++i) {
                    a.x = fmaf(pp[i], vx[i].x, a.x); a.y = fmaf(pp[i], vx[i].y, a.y);
                    a.z = fmaf(pp[i], vx[i].z, a.z); a.w = fmaf(pp[i], vx[i].w, a.w);
                }
                acc[r] = a;
            }
        }
    }

#pragma unroll
    for (int r = 0; r < MR; ++r)
        if (r < n_rows) *reinterpret_cast<float4*>(&part_acc[w][r][lane * 4]) = acc[r];
    if (pi == 0) {
#pragma unroll
        for (int t = 0; t < N3; ++t) part_ml[w][row_base + t] = make_float2(m_own[t], l_own[t]);
    }
    __syncthreads();
    for (int r = 0; r < n_rows; ++r) {                      // thread d merges the four warps in warp order
        float M = -INFINITY;
#pragma unroll
        for (int ww = 0; ww < NW; ++ww) M = fmaxf(M, part_ml[ww][r].x);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int ww = 0; ww < NW; ++ww) {
            const float2 ml = part_ml[ww][r];
            const float wt = (ml.x == -INFINITY) ? 0.f : expf(ml.x - M);
            num = fmaf(wt, part_acc[ww][r][tid], num);
            den = fmaf(wt, ml.y, den);
        }
        o_part[(((size_t)h * max_splits + s) * ROWS + row0 + r) * DH + tid] = num;
        if (tid == 0) ml_part[((size_t)h * max_splits + s) * ROWS + row0 + r] = make_float2(M, den);
    }

    // One-row forwards (draft and vanilla steps) merge the chunks here instead of in a launch of their own: every
    // CTA of the head arrives on a counter once its partial result is stored, and the last one to arrive runs the
    // same merge the combine kernel runs (zero on entry, zero again on exit; dynamic smem = 2 * max_splits floats).
    if constexpr (MR == 1) {
        if (head_counters) {
            __shared__ int last_sh;
            __shared__ float wmax_sh[32];
            extern __shared__ float comb_sh[];
            __syncthreads();                                    // this CTA's stores precede its arrival
            if (tid == 0) {
                const int n_chunks = (total + ATTN_CHUNK - 1) / ATTN_CHUNK;
                last_sh = atom_add_acq_rel_gpu(&head_counters[h], 1) == n_chunks - 1;
            }
            __syncthreads();
            if (last_sh) {
                combine_row(pos0, 0, h, o_part, ml_part, max_splits, n_heads, DH, out, planes, comb_sh, wmax_sh);
                if (tid == 0) head_counters[h] = 0;
            }
        }
    }
}

// grid = (H, rows), block = dh threads, dynamic smem = 2 * max_splits floats.  Combines the splits in chunk
// order (combine_row above).
__global__ void attn_combine_kernel(const DevState* st, const float* __restrict__ o_part,
                                    const float2* __restrict__ ml_part, int max_splits, int n_heads, int dh,
                                    float* __restrict__ out, __nv_bfloat16* __restrict__ planes, int part_rows,
                                    int row_base, int n_rows_fixed, int pos0_fixed, int n_seq)
{
    // row_base / n_rows_fixed / pos0_fixed: as in attn_mma_kernel (one sequence inside a larger chunk), 0 / 0 / 0 otherwise;
    // n_seq > 1: grid.y covers that many such sequences, one after another
    pdl_enter();
    int r = blockIdx.y;
    if (n_seq > 1) {
        const int seq = r / n_rows_fixed;
        if (seq >= n_seq) return;
        r -= seq * n_rows_fixed;
        row_base += seq * n_rows_fixed;
    }
    if (r >= (n_rows_fixed > 0 ? n_rows_fixed : st->n_rows)) return;
    extern __shared__ float comb_sh[];
    __shared__ float wmax_sh[32];
    combine_row(n_rows_fixed > 0 ? pos0_fixed : st->pos0, r, blockIdx.x, o_part, ml_part, max_splits, n_heads, dh, out, planes, comb_sh,
                wmax_sh, part_rows, row_base);
}

} // namespace swk
