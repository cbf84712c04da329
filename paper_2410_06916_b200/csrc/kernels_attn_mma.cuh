// Attention of the target model's forwards (verification of the drafted rows, vanilla steps, prefill chunks) on the
// tensor cores: softmax(q K^T / sqrt(d_h)) V over the paged cache for head_dim 128, split over 64-position chunks
// like the streaming kernel next door and merged by the same combine step.
//
// One CTA = one KV head x one chunk, for ALL query heads of that KV head's group and all rows of the forward
// (R = group size x rows "query rows"), so a K/V byte is loaded once per forward however many heads share it.
// The contraction is issued "swapped", with the streamed operand on the M side of mma.sync.m16n8k16 (bf16):
//     S^T [16 positions x 8 query rows] = K [16 positions x 128 dims]   . Q^T [128 dims x 8 query rows]
//     O^T [16 dims      x 8 query rows] = V^T [16 dims x 16 positions]  . P^T [16 positions x 8 query rows]
// so accumulator registers scale with the number of query rows (one 8-row tile for a one-row forward, two for a
// verification) and K, V go from global memory straight into A fragments: the k index of a contraction may be
// permuted freely as long as both operands agree, so every lane loads 16-byte pieces (K: lane (g, t) takes dims
// 16j + 4t .. +3 of positions g and g + 8; V: dims 32i + 4g .. +3 of positions t, t + 4, t + 8, t + 12) and the
// fragment elements are picked out of them, no shuffle and no shared-memory staging.  Warp w owns positions
// [16w, 16w + 16) of the chunk; the four warps' partial results are merged in warp order.
//
// Precision: cached K,V and the queries are fp32.  Every operand is split into two bf16 numbers, hi = bf16(x) and
// lo = bf16(x - hi) (16 significant bits together, the same treatment the weight-streaming GEMM gives its
// activations), and a product is three MMAs (lo*hi, hi*lo, hi*hi); accumulation is fp32.  (The tf32 form of the
// same kernel, m16n8k8 with four times as many MMA instructions, was bound by the issue rate of the legacy tensor
// path and slower than the FMA kernel it was meant to replace.)
//
// Which rows a query row sees among the forward's own rows comes from a bit mask per row in the control block
// (plain causal order, or the ancestors of a node when a token tree is verified); cached positions below the
// forward's first row are visible to all.  A row's result depends on neither the other rows nor their number.
#pragma once
#include "common.cuh"
#include "kernels_attn.cuh"

namespace swk {

constexpr int AM_THREADS = 128;
#ifndef SWIFT_AM_V_LATE
#define SWIFT_AM_V_LATE 1
#endif
#ifndef SWIFT_AM_CTAS
#define SWIFT_AM_CTAS 3
#endif
constexpr bool AM_V_LATE = SWIFT_AM_V_LATE != 0;   // V loaded after the scores (fewer live registers, more CTAs per SM)
constexpr int AM_QSTRIDE = 144;     // bf16 per staged query row (288 bytes): the rows of a fragment load fall into different banks
constexpr int AM_OSTRIDE = 132;     // floats per row of a warp's partial output
constexpr int AM_PSTRIDE = 20;      // floats per row of a warp's probabilities (16 positions)

__host__ __device__ constexpr size_t attn_mma_smem_bytes(int nt, int max_splits)
{
    return (size_t)(2 * 8 * nt * AM_QSTRIDE) * 2 +
           (size_t)(4 * 8 * nt * AM_OSTRIDE + 4 * 8 * nt * AM_PSTRIDE + 2 * 4 * 8 * nt + 2 * max_splits) * 4;
}

// Two fp32 numbers -> their bf16 hi parts and lo parts, each pair packed into one register (first number in the
// low half, as the MMA fragments want it): hi = bf16(x), lo = bf16(x - hi), both rounded to nearest.
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t& hi, uint32_t& lo)
{
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(x1), "f"(x0));
    const float r0 = x0 - __uint_as_float(hi << 16), r1 = x1 - __uint_as_float(hi & 0xFFFF0000u);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(r1), "f"(r0));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// c += a * b with both operands given as hi + lo: the small terms first
__device__ __forceinline__ void mma_split(float (&c)[4], const uint32_t (&ah)[4], const uint32_t (&al)[4], uint32_t bh0,
                                          uint32_t bh1, uint32_t bl0, uint32_t bl1)
{
    mma_bf16(c, al, bh0, bh1);
    mma_bf16(c, ah, bl0, bl1);
    mma_bf16(c, ah, bh0, bh1);
}

// grid = (n_kv_heads, max_splits), block = 128, dynamic smem = attn_mma_smem_bytes(NT, max_splits).
// NT = 8-row tiles of query rows processed together (1: up to 8 query rows per pass, 2: up to 16); more query rows
// are taken in several passes, each of which fetches the warp's K,V pieces again (from L1/L2 after the first).
// part_rows = row stride of o_part / ml_part: o_part[h][s][part_rows][128] (unnormalised), ml_part[h][s][part_rows].
// head_counters / out / planes: as in attn_stream_kernel, used for one-row forwards only (merge by the last CTA).
template <typename T, int NT>
__global__ void __launch_bounds__(AM_THREADS, SWIFT_AM_CTAS)
attn_mma_kernel(const DevState* st, const float* __restrict__ q, const T* __restrict__ kv_pool,
                const int* __restrict__ page_table, KvLayout L, int block, int n_heads, int max_splits, float scale,
                float* __restrict__ o_part, float2* __restrict__ ml_part, int part_rows, int* __restrict__ head_counters,
                float* __restrict__ out, __nv_bfloat16* __restrict__ planes, int row_base, int n_rows_fixed, int pos0_fixed)
{
    // n_rows_fixed > 0: the rows [row_base, row_base + n_rows_fixed) of a larger chunk form one sequence of their own, whose
    // first row sits at cache slot pos0_fixed (candidate scoring); otherwise the whole forward is the sequence.
    pdl_enter();
    constexpr int DH = 128, QR = 8 * NT;                    // query rows per pass
    const int n_rows = n_rows_fixed > 0 ? n_rows_fixed : st->n_rows;
    if (n_rows <= 0) return;
    const int pos0 = n_rows_fixed > 0 ? pos0_fixed : st->pos0, total = pos0 + n_rows;
    q += (size_t)row_base * n_heads * 128;
    const int kvh = blockIdx.x, s = blockIdx.y, c0 = s * ATTN_CHUNK;
    if (c0 >= total) return;
    const int len = min(ATTN_CHUNK, total - c0);
    const int G = n_heads / L.n_kv_heads, R = G * n_rows;   // query row rho = hl * n_rows + r: head hl of the group, row r
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, g = lane >> 2, t = lane & 3;
    const int j0 = w * 16;
    const bool live = j0 < len;                             // this warp's 16 positions hold something

    extern __shared__ __align__(16) float am_smem[];
    __nv_bfloat16* q_hi = reinterpret_cast<__nv_bfloat16*>(am_smem);   // [QR][AM_QSTRIDE]
    __nv_bfloat16* q_lo = q_hi + QR * AM_QSTRIDE;
    float* part_acc = reinterpret_cast<float*>(q_lo + QR * AM_QSTRIDE);   // [4][QR][AM_OSTRIDE]
    float* p_sh = part_acc + 4 * QR * AM_OSTRIDE;           // [4][QR][AM_PSTRIDE]
    float2* part_ml = reinterpret_cast<float2*>(p_sh + 4 * QR * AM_PSTRIDE);   // [4][QR]
    float* comb_sh = reinterpret_cast<float*>(part_ml + 4 * QR);               // [2 * max_splits]
    __shared__ unsigned vis_sh[ROWS];
    if (tid < ROWS) vis_sh[tid] = st->row_vis[tid];

    // where this warp's K and V pieces live (rows past the end re-read the last one; they are masked below)
    const T *ka = kv_pool, *kb = kv_pool, *vp[4] = {kv_pool, kv_pool, kv_pool, kv_pool};
    if (live) {
        const int pa = c0 + min(j0 + g, len - 1), pb = c0 + min(j0 + g + 8, len - 1);
        ka = kv_pool + L.offset(__ldg(page_table + (pa >> L.page_shift)), block, 0, kvh, pa & (L.page_size - 1)) + 4 * t;
        kb = kv_pool + L.offset(__ldg(page_table + (pb >> L.page_shift)), block, 0, kvh, pb & (L.page_size - 1)) + 4 * t;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int pv = c0 + min(j0 + t + 4 * u, len - 1);
            vp[u] = kv_pool + L.offset(__ldg(page_table + (pv >> L.page_shift)), block, 1, kvh, pv & (L.page_size - 1)) + 4 * g;
        }
    }

    const int n_pass = (R + QR - 1) / QR;
    // gridDim.z > 1: the passes are spread over the grid's z dimension, one per CTA (chunks of many rows: the first
    // chunks of a prompt have few K,V chunks and would otherwise leave most SMs idle)
    const int pass_begin = gridDim.z > 1 ? (int)blockIdx.z : 0;
    const int pass_end = gridDim.z > 1 ? min(n_pass, (int)blockIdx.z + 1) : n_pass;
#pragma unroll 1
    for (int pass = pass_begin; pass < pass_end; ++pass) {
        const int rho0 = pass * QR;
        {   // a pass none of whose rows sees this chunk yet (causal order) has nothing to add: the merge never reads it
            const int rho1 = min(R, rho0 + QR) - 1;
            const int r_last = (rho0 / n_rows == rho1 / n_rows) ? rho1 % n_rows : n_rows - 1;
            if (n_rows > ROWS && c0 > pos0 + r_last) continue;
        }
        // K and V go from memory straight into fragment order, once per pass: a forward with more query rows than one
        // pass takes (grouped-query models) reads them again from L1/L2 rather than holding 128 registers of them
        // across the loop.  The empty asm keeps the compiler from hoisting the loads (and their hi/lo splits) out of it.
        float4 kA[8], kB[8], vv[4][4];
        if (live) {
            asm volatile("" : "+l"(ka), "+l"(kb));
#pragma unroll
            for (int j = 0; j < 8; ++j) { kA[j] = load_row4<T>(ka + 16 * j); kB[j] = load_row4<T>(kb + 16 * j); }
            if (!AM_V_LATE) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    asm volatile("" : "+l"(vp[u]));
#pragma unroll
                    for (int i = 0; i < 4; ++i) vv[u][i] = load_row4<T>(vp[u] + 32 * i);
                }
            }
        }
        __syncthreads();                                    // the previous pass's merge has read part_acc; vis_sh is set
        // ---- stage this pass's query rows, scaled and split
        for (int i = tid; i < QR * 32; i += AM_THREADS) {
            const int rl = i >> 5, c4 = i & 31, rho = rho0 + rl;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (rho < R) {
                const int hl = rho / n_rows, r = rho - hl * n_rows;
                v = *reinterpret_cast<const float4*>(q + ((size_t)r * n_heads + kvh * G + hl) * DH + c4 * 4);
                v.x *= scale; v.y *= scale; v.z *= scale; v.w *= scale;
            }
            uint2 hi, lo;
            split_pair(v.x, v.y, hi.x, lo.x);
            split_pair(v.z, v.w, hi.y, lo.y);
            *reinterpret_cast<uint2*>(q_hi + rl * AM_QSTRIDE + c4 * 4) = hi;
            *reinterpret_cast<uint2*>(q_lo + rl * AM_QSTRIDE + c4 * 4) = lo;
        }
        __syncthreads();

        if (live) {
            // ---- scores: sacc[nt][0], [1] = (position j0 + g, query rows 8nt + 2t, + 1); [2], [3] = position j0 + g + 8
            float sacc[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) { sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f; }
#pragma unroll
            for (int j = 0; j < 8; ++j) {                   // k-step j: dims 16j .. 16j + 15, this lane's share 16j + 4t .. + 3
                uint32_t ah[4], al[4];
                split_pair(kA[j].x, kA[j].y, ah[0], al[0]); split_pair(kB[j].x, kB[j].y, ah[1], al[1]);
                split_pair(kA[j].z, kA[j].w, ah[2], al[2]); split_pair(kB[j].z, kB[j].w, ah[3], al[3]);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint2 bh = *reinterpret_cast<const uint2*>(q_hi + (8 * nt + g) * AM_QSTRIDE + 16 * j + 4 * t);
                    const uint2 bl = *reinterpret_cast<const uint2*>(q_lo + (8 * nt + g) * AM_QSTRIDE + 16 * j + 4 * t);
                    mma_split(sacc[nt], ah, al, bh.x, bh.y, bl.x, bl.y);
                }
            }

            if (AM_V_LATE) {                                // V is requested once K's registers are free: the soft-max covers part of the wait
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    asm volatile("" : "+l"(vp[u]));
#pragma unroll
                    for (int i = 0; i < 4; ++i) vv[u][i] = load_row4<T>(vp[u] + 32 * i);
                }
            }
            // ---- soft-max over this warp's 16 positions, per query row (the 8 lanes that share t hold one row's scores)
            float* pw = p_sh + w * QR * AM_PSTRIDE;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int rl = 8 * nt + 2 * t + e, rho = rho0 + rl;
                    float x0 = -INFINITY, x1 = -INFINITY;
                    if (rho < R) {
                        const int r = rho % n_rows;
                        const int p0 = c0 + j0 + g, p1 = p0 + 8;
                        // a position is visible when it is cached context, or one of the forward's rows this row may see
                        auto visible = [&](int p) -> bool {
                            if (p >= total) return false;
                            if (p < pos0) return true;
                            const int dlt = p - pos0;
                            return n_rows <= ROWS ? ((vis_sh[r] >> dlt) & 1u) != 0u : dlt <= r;
                        };
                        if (visible(p0)) x0 = sacc[nt][e];
                        if (visible(p1)) x1 = sacc[nt][2 + e];
                    }
                    float m = fmaxf(x0, x1);
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
                    const float e0 = (x0 == -INFINITY) ? 0.f : expf(x0 - m);
                    const float e1 = (x1 == -INFINITY) ? 0.f : expf(x1 - m);
                    float l = e0 + e1;
                    l += __shfl_xor_sync(0xffffffffu, l, 4);
                    l += __shfl_xor_sync(0xffffffffu, l, 8);
                    l += __shfl_xor_sync(0xffffffffu, l, 16);
                    pw[rl * AM_PSTRIDE + g] = e0;
                    pw[rl * AM_PSTRIDE + g + 8] = e1;
                    if (g == 0) part_ml[w * QR + rl] = make_float2(m, l);
                }
            }
            __syncwarp();

            // ---- outputs: oacc[nt][2i + hf] = (dims 32i + 4g + 2hf, + 1) x (query rows 8nt + 2t, + 1)
            float oacc[NT][8][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) { oacc[nt][mt][0] = oacc[nt][mt][1] = oacc[nt][mt][2] = oacc[nt][mt][3] = 0.f; }
            {                                               // one k-step: the warp's 16 positions, this lane's share t, t + 4, t + 8, t + 12
                uint32_t bh0[NT], bh1[NT], bl0[NT], bl1[NT];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const float* pr = pw + (8 * nt + g) * AM_PSTRIDE + t;
                    split_pair(pr[0], pr[4], bh0[nt], bl0[nt]);
                    split_pair(pr[8], pr[12], bh1[nt], bl1[nt]);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t ah[4], al[4];
                    split_pair(vv[0][i].x, vv[1][i].x, ah[0], al[0]); split_pair(vv[0][i].y, vv[1][i].y, ah[1], al[1]);
                    split_pair(vv[2][i].x, vv[3][i].x, ah[2], al[2]); split_pair(vv[2][i].y, vv[3][i].y, ah[3], al[3]);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_split(oacc[nt][2 * i], ah, al, bh0[nt], bh1[nt], bl0[nt], bl1[nt]);
                    split_pair(vv[0][i].z, vv[1][i].z, ah[0], al[0]); split_pair(vv[0][i].w, vv[1][i].w, ah[1], al[1]);
                    split_pair(vv[2][i].z, vv[3][i].z, ah[2], al[2]); split_pair(vv[2][i].w, vv[3][i].w, ah[3], al[3]);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_split(oacc[nt][2 * i + 1], ah, al, bh0[nt], bh1[nt], bl0[nt], bl1[nt]);
                }
            }
            float* ow = part_acc + (size_t)w * QR * AM_OSTRIDE;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    *reinterpret_cast<float4*>(ow + (8 * nt + 2 * t) * AM_OSTRIDE + 32 * i + 4 * g) =
                        make_float4(oacc[nt][2 * i][0], oacc[nt][2 * i][2], oacc[nt][2 * i + 1][0], oacc[nt][2 * i + 1][2]);
                    *reinterpret_cast<float4*>(ow + (8 * nt + 2 * t + 1) * AM_OSTRIDE + 32 * i + 4 * g) =
                        make_float4(oacc[nt][2 * i][1], oacc[nt][2 * i][3], oacc[nt][2 * i + 1][1], oacc[nt][2 * i + 1][3]);
                }
        } else if (lane < QR) {
            part_ml[w * QR + lane] = make_float2(-INFINITY, 0.f);   // nothing here: the merge leaves this warp out
        }
        __syncthreads();

        // ---- merge the four warps in warp order: thread d takes dimension d of every query row of the pass
        const int n_live = min(4, (len + 15) >> 4);
        for (int rl = 0; rl < QR && rho0 + rl < R; ++rl) {
            const int rho = rho0 + rl, hl = rho / n_rows, r = rho - hl * n_rows;
            float M = -INFINITY;
            for (int ww = 0; ww < n_live; ++ww) M = fmaxf(M, part_ml[ww * QR + rl].x);
            float num = 0.f, den = 0.f;
            for (int ww = 0; ww < n_live; ++ww) {
                const float2 ml = part_ml[ww * QR + rl];
                if (ml.x == -INFINITY) continue;
                const float wt = expf(ml.x - M);
                num = fmaf(wt, part_acc[((size_t)ww * QR + rl) * AM_OSTRIDE + tid], num);
                den = fmaf(wt, ml.y, den);
            }
            const size_t slot = ((size_t)(kvh * G + hl) * max_splits + s) * part_rows + row_base + r;
            o_part[slot * DH + tid] = num;
            if (tid == 0) ml_part[slot] = make_float2(M, den);
        }
    }

    // One-row forwards (vanilla steps) merge the chunks here: the last CTA of a KV head to arrive on its counter runs
    // the combine step for the group's heads (counter zero on entry and again on exit).
    if (head_counters != nullptr && n_rows == 1) {
        __shared__ int last_sh;
        __shared__ float wmax_sh[32];
        __syncthreads();
        if (tid == 0) {
            const int n_chunks = (total + ATTN_CHUNK - 1) / ATTN_CHUNK;
            last_sh = atom_add_acq_rel_gpu(&head_counters[kvh], 1) == n_chunks - 1;
        }
        __syncthreads();
        if (last_sh) {
            for (int hl = 0; hl < G; ++hl) {
                combine_row(pos0, 0, kvh * G + hl, o_part, ml_part, max_splits, n_heads, DH, out, planes, comb_sh, wmax_sh, part_rows);
                __syncthreads();
            }
            if (tid == 0) head_counters[kvh] = 0;
        }
    }
}

} // namespace swk
