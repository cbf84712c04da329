// Attention for chunks of many rows (prefill chunks, the window rows of a scored candidate): one CTA = one KV head x one
// 64-position chunk of the cache x up to four tiles of 64 query rows, taken in turn (query row rho = hl * n_rows + r: head hl of the KV head's
// group, row r of the sequence).  The chunk's K and V are loaded from the paged cache once per CTA, split into
// bf16 hi / lo planes (16 significant bits together, as everywhere else) and kept in shared memory; each of the four
// warps owns 16 query rows and runs S = Q K^T and O = P V on mma.sync.m16n8k16 with three MMAs per product
// (lo*hi, hi*lo, hi*hi), fp32 accumulation, a soft-max over the chunk per row in registers.  Outputs are the same
// unnormalised partial results per (head, chunk, row) that the other attention kernels write; the combine step merges
// the chunks.  Visibility: cached context below the sequence's first row, then causal order among its rows.
#pragma once
#include "common.cuh"
#include "kernels_attn_mma.cuh"

namespace swk {

constexpr int AT_THREADS = 128;
constexpr int AT_QROWS = 64;            // query rows per tile (16 per warp)
constexpr int AT_TPC = 4;               // tiles a CTA takes in turn on one staged chunk
constexpr int AT_KSTRIDE = 136;         // bf16 per staged K or V row (128 + 8: rows of a fragment load fall into different banks)
constexpr size_t AT_SMEM_BYTES = (size_t)4 * ATTN_CHUNK * AT_KSTRIDE * 2;   // K hi, K lo, V hi, V lo

__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t& r0, uint32_t& r1, const void* row_ptr)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(row_ptr);
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(a));
}

// grid = (n_kv_heads, max_splits, ceil(query tiles / AT_TPC)), block = 128, dynamic smem = AT_SMEM_BYTES.
// row_base / n_rows_fixed / pos0_fixed: as in attn_mma_kernel (a sequence inside a larger chunk), else 0 / 0 / 0.
// n_seq > 1: that many such sequences in one launch (grid.z covers the larger of the batch's and the sequences' tiles),
// page tables pt_stride ints apart.
template <typename T>
__global__ void __launch_bounds__(AT_THREADS, 2)
attn_tile_kernel(const DevState* st, const float* __restrict__ q, const T* __restrict__ kv_pool,
                 const int* __restrict__ page_table, KvLayout L, int block, int n_heads, int max_splits, float scale,
                 float* __restrict__ o_part, float2* __restrict__ ml_part, int part_rows, int row_base, int n_rows_fixed,
                 int pos0_fixed, int n_seq, int pt_stride)
{
    pdl_enter();
    constexpr int DH = 128;
    int n_rows = n_rows_fixed > 0 ? n_rows_fixed : st->n_rows;
    if (n_rows <= 0) return;
    const int pos0 = n_rows_fixed > 0 ? pos0_fixed : st->pos0, total = pos0 + n_rows;
    const int kvh = blockIdx.x, s = blockIdx.y, c0 = s * ATTN_CHUNK;
    if (c0 >= total) return;
    const int len = min(ATTN_CHUNK, total - c0);
    const int G = n_heads / L.n_kv_heads;
    int z = blockIdx.z;
    bool per_seq = false;
    if (n_seq > 1) {
        // n_seq sequences of n_rows rows side by side (rows row_base + seq * n_rows ..), all continuing the same cached
        // context, each with its own page table for its own rows.  A chunk that lies inside the context is the same for
        // all of them and fully visible to every row: it is staged once per 64 rows of the whole batch.  A chunk that
        // reaches into the sequences' own rows is handled per sequence.
        if (c0 + ATTN_CHUNK <= pos0) {
            n_rows *= n_seq;
        } else {
            const int tiles_per = (G * n_rows + AT_QROWS - 1) / AT_QROWS, seq = z / tiles_per;
            if (seq >= n_seq) return;
            per_seq = true;
            z -= seq * tiles_per;
            row_base += seq * n_rows;
            page_table += (size_t)seq * pt_stride;
        }
    }
    const int R = G * n_rows;
    // the CTA stages its chunk once and then takes up to AT_TPC tiles of 64 query rows in turn (one tile where every sequence
    // has a chunk of its own)
    const int tile_first = per_seq ? z : z * AT_TPC, tile_count = per_seq ? 1 : AT_TPC;
    if (tile_first * AT_QROWS >= R) return;
    {   // tiles none of whose rows sees this chunk yet have nothing to add: the merge never reads them
        const int rho0 = tile_first * AT_QROWS, rho1 = min(R, (tile_first + tile_count) * AT_QROWS) - 1;
        const int r_last = (rho0 / n_rows == rho1 / n_rows) ? rho1 % n_rows : n_rows - 1;
        if (c0 > pos0 + r_last) return;
    }
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, g = lane >> 2, t = lane & 3;
    q += (size_t)row_base * n_heads * DH;

    extern __shared__ __align__(16) unsigned char at_smem[];
    __nv_bfloat16* k_hi = reinterpret_cast<__nv_bfloat16*>(at_smem);          // [64][AT_KSTRIDE]
    __nv_bfloat16* k_lo = k_hi + ATTN_CHUNK * AT_KSTRIDE;
    __nv_bfloat16* v_hi = k_lo + ATTN_CHUNK * AT_KSTRIDE;
    __nv_bfloat16* v_lo = v_hi + ATTN_CHUNK * AT_KSTRIDE;

    // ---- stage the chunk: thread i takes 16-byte pieces (4 dims of one position); positions past the end are zero.
    // The pages of the chunk's positions are looked up first and the loads of eight pieces are issued together, so that
    // a CTA waits for two or three trips to memory rather than for one per piece.
    __shared__ int page_of[ATTN_CHUNK];
    if (tid < ATTN_CHUNK) page_of[tid] = tid < len ? __ldg(page_table + ((c0 + tid) >> L.page_shift)) : 0;

    __syncthreads();
#pragma unroll
    for (int part = 0; part < ATTN_CHUNK * 32 / (8 * AT_THREADS); ++part) {
        float4 kk[8], vv[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int i = tid + (part * 8 + it) * AT_THREADS, p = i >> 5, c4 = (i & 31) * 4;
            kk[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            vv[it] = kk[it];
            if (p < len) {
                const int slot = (c0 + p) & (L.page_size - 1);
                kk[it] = load_row4<T>(kv_pool + L.offset(page_of[p], block, 0, kvh, slot) + c4);
                vv[it] = load_row4<T>(kv_pool + L.offset(page_of[p], block, 1, kvh, slot) + c4);
            }
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int i = tid + (part * 8 + it) * AT_THREADS, p = i >> 5, c4 = (i & 31) * 4;
            uint2 hi, lo;
            split_pair(kk[it].x, kk[it].y, hi.x, lo.x); split_pair(kk[it].z, kk[it].w, hi.y, lo.y);
            *reinterpret_cast<uint2*>(k_hi + p * AT_KSTRIDE + c4) = hi;
            *reinterpret_cast<uint2*>(k_lo + p * AT_KSTRIDE + c4) = lo;
            split_pair(vv[it].x, vv[it].y, hi.x, lo.x); split_pair(vv[it].z, vv[it].w, hi.y, lo.y);
            *reinterpret_cast<uint2*>(v_hi + p * AT_KSTRIDE + c4) = hi;
            *reinterpret_cast<uint2*>(v_lo + p * AT_KSTRIDE + c4) = lo;
        }
    }
    __syncthreads();

    for (int ti = 0; ti < tile_count; ++ti) {              // no barrier below: the warps go through their tiles on their own
    const int rho_tile = (tile_first + ti) * AT_QROWS;
    if (rho_tile >= R) break;
    {
        const int rho1 = min(R, rho_tile + AT_QROWS) - 1;
        const int r_last = (rho_tile / n_rows == rho1 / n_rows) ? rho1 % n_rows : n_rows - 1;
        if (c0 > pos0 + r_last) continue;                   // this tile sees nothing of the chunk
    }
    // ---- this warp's 16 query rows as A fragments (hi, lo), scaled: rows rho_w + g and rho_w + g + 8
    const int rho_w = rho_tile + 16 * w;
    if (rho_w >= R) break;
    const int rho_a = rho_w + g, rho_b = rho_w + g + 8;
    const bool live_a = rho_a < R, live_b = rho_b < R;
    const int hl_a = live_a ? rho_a / n_rows : 0, r_a = live_a ? rho_a - hl_a * n_rows : 0;
    const int hl_b = live_b ? rho_b / n_rows : 0, r_b = live_b ? rho_b - hl_b * n_rows : 0;
    const float* qa = q + ((size_t)r_a * n_heads + kvh * G + hl_a) * DH;
    const float* qb = q + ((size_t)r_b * n_heads + kvh * G + hl_b) * DH;
    uint32_t qh[8][4], ql[8][4];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {                        // k-step ks: dims 16 ks .. 16 ks + 15
        float2 a0 = make_float2(0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;
        if (live_a) { a0 = *reinterpret_cast<const float2*>(qa + 16 * ks + 2 * t); a2 = *reinterpret_cast<const float2*>(qa + 16 * ks + 8 + 2 * t); }
        if (live_b) { a1 = *reinterpret_cast<const float2*>(qb + 16 * ks + 2 * t); a3 = *reinterpret_cast<const float2*>(qb + 16 * ks + 8 + 2 * t); }
        split_pair(a0.x * scale, a0.y * scale, qh[ks][0], ql[ks][0]);
        split_pair(a1.x * scale, a1.y * scale, qh[ks][1], ql[ks][1]);
        split_pair(a2.x * scale, a2.y * scale, qh[ks][2], ql[ks][2]);
        split_pair(a3.x * scale, a3.y * scale, qh[ks][3], ql[ks][3]);
    }

    // ---- scores of the warp's 16 rows against the chunk's 64 positions: 8 tiles of 8 positions
    float sacc[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) { sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const __nv_bfloat16* kr = k_hi + (8 * nt + g) * AT_KSTRIDE + 16 * ks + 2 * t;
            const uint32_t bh0 = *reinterpret_cast<const uint32_t*>(kr), bh1 = *reinterpret_cast<const uint32_t*>(kr + 8);
            const __nv_bfloat16* kl = k_lo + (8 * nt + g) * AT_KSTRIDE + 16 * ks + 2 * t;
            const uint32_t bl0 = *reinterpret_cast<const uint32_t*>(kl), bl1 = *reinterpret_cast<const uint32_t*>(kl + 8);
            mma_split(sacc[nt], qh[ks], ql[ks], bh0, bh1, bl0, bl1);
        }
    }

    // ---- mask and soft-max over the chunk, per row (row g in elements 0, 1; row g + 8 in elements 2, 3)
    float m_a = -INFINITY, m_b = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int p = c0 + 8 * nt + 2 * t + e;          // visible: cached context, or a row of the sequence not after this one
            if (!(live_a && (p < pos0 || p - pos0 <= r_a))) sacc[nt][e] = -INFINITY;
            if (!(live_b && (p < pos0 || p - pos0 <= r_b))) sacc[nt][2 + e] = -INFINITY;
            m_a = fmaxf(m_a, sacc[nt][e]);
            m_b = fmaxf(m_b, sacc[nt][2 + e]);
        }
    m_a = fmaxf(m_a, __shfl_xor_sync(0xffffffffu, m_a, 1)); m_a = fmaxf(m_a, __shfl_xor_sync(0xffffffffu, m_a, 2));
    m_b = fmaxf(m_b, __shfl_xor_sync(0xffffffffu, m_b, 1)); m_b = fmaxf(m_b, __shfl_xor_sync(0xffffffffu, m_b, 2));
    float l_a = 0.f, l_b = 0.f;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float pa = sacc[nt][e] == -INFINITY ? 0.f : expf(sacc[nt][e] - m_a);
            const float pb = sacc[nt][2 + e] == -INFINITY ? 0.f : expf(sacc[nt][2 + e] - m_b);
            sacc[nt][e] = pa; sacc[nt][2 + e] = pb;
            l_a += pa; l_b += pb;
        }
    l_a += __shfl_xor_sync(0xffffffffu, l_a, 1); l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
    l_b += __shfl_xor_sync(0xffffffffu, l_b, 1); l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);

    // ---- outputs: O[16 rows][128 dims] = P[16 x 64] V[64 x 128]; the probabilities are already in A-fragment order
    float oacc[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { oacc[nt][0] = oacc[nt][1] = oacc[nt][2] = oacc[nt][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {                        // positions 16 kk .. 16 kk + 15
        uint32_t ph[4], pl[4];
        split_pair(sacc[2 * kk][0], sacc[2 * kk][1], ph[0], pl[0]);
        split_pair(sacc[2 * kk][2], sacc[2 * kk][3], ph[1], pl[1]);
        split_pair(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1], ph[2], pl[2]);
        split_pair(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3], ph[3], pl[3]);
        const int vrow = 16 * kk + (lane & 15);             // ldmatrix row addresses: positions 16 kk + 0..15
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {                   // dims 8 nt .. 8 nt + 7
            uint32_t bh0, bh1, bl0, bl1;
            ldmatrix_x2_trans(bh0, bh1, v_hi + vrow * AT_KSTRIDE + 8 * nt);
            ldmatrix_x2_trans(bl0, bl1, v_lo + vrow * AT_KSTRIDE + 8 * nt);
            mma_split(oacc[nt], ph, pl, bh0, bh1, bl0, bl1);
        }
    }

    // ---- partial results of this chunk: unnormalised outputs, running maximum and sum per row
    if (live_a) {
        const size_t slot = ((size_t)(kvh * G + hl_a) * max_splits + s) * part_rows + row_base + r_a;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
            *reinterpret_cast<float2*>(o_part + slot * DH + 8 * nt + 2 * t) = make_float2(oacc[nt][0], oacc[nt][1]);
        if (t == 0) ml_part[slot] = make_float2(m_a, l_a);
    }
    if (live_b) {
        const size_t slot = ((size_t)(kvh * G + hl_b) * max_splits + s) * part_rows + row_base + r_b;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
            *reinterpret_cast<float2*>(o_part + slot * DH + 8 * nt + 2 * t) = make_float2(oacc[nt][2], oacc[nt][3]);
        if (t == 0) ml_part[slot] = make_float2(m_b, l_b);
    }
    }
}

} // namespace swk
