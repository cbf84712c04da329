// Element-wise and per-row kernels of the decoder walk: state set-up, embedding gather,
// residual-add + RMSNorm, RoPE + KV append, SwiGLU.  All of them take their row count and base
// position from the device-resident DevState and do nothing when it holds zero rows.
#pragma once
#include "common.cuh"
#include "kernels_gemm_tc.cuh"

namespace swk {

// ------------------------------------------------------------------------------ state
// Generic forward chunk: tokens were copied into st->row_tok beforehand.
__global__ void set_rows_kernel(DevState* st, int pos0, int n_rows)
{
    st->pos0 = pos0;
    st->n_rows = n_rows;
    st->tok_off = 0;
    set_causal_rows(st);
}

// Start of a round: pending token into slot 0, drafting armed.
__global__ void begin_round_kernel(DevState* st, int pending_token, int use_given_token, int round, float stop_conf,
                                   unsigned seed_lo, unsigned seed_hi)
{
    if (use_given_token) st->draft_tok[0] = pending_token;
    st->round = round;
    st->stop_conf = stop_conf;
    st->seed_lo = seed_lo;
    st->seed_hi = seed_hi;
    st->active = 1;
    st->n_drafted = 0;
    st->n_accepted = 0;
    set_causal_rows(st);
}

// Draft step j (1-based): one row, input y'_{j-1} (slot j-1), position n + j - 1; a stopped draft
// leaves zero rows so that the step's kernels fall through.
__global__ void begin_draft_step_kernel(DevState* st, int n, int j)
{
    st->draft_j = j;
    if (st->active) {
        st->pos0 = n + j - 1;
        st->n_rows = 1;
        st->tok_off = j - 1;
    } else {
        st->n_rows = 0;
    }
}

// Verification: rows [t*, y'_1..y'_k] with k taken from the device (or forced by the host).
__global__ void begin_verify_kernel(DevState* st, int n, int forced_k)
{
    if (forced_k >= 0) st->n_drafted = forced_k;
    set_causal_rows(st);
    st->pos0 = n;
    st->n_rows = st->n_drafted + 1;
    st->tok_off = 0;
}

// How many of the draft model's top predictions stand in for a draft token of confidence p (Section 4.2):
// 10, 5, 3, 1 for p in (0, 0.5], (0.5, 0.8], (0.8, 0.95], (0.95, 1].
__host__ __device__ inline int tree_width(float p) { return p <= 0.5f ? 10 : p <= 0.8f ? 5 : p <= 0.95f ? 3 : 1; }

// Verification of a token tree built on the device: rows 0..k are the chain [t*, y'_1..y'_k] as in a plain
// verification; the remaining rows (up to `budget` in all) hold, draft position by draft position from the first on,
// the next-best predictions the draft model made there (cand[(j-1)*TREE_TOPK + i], i >= 1; cand_n[j-1] of them count,
// the chain token included).  An alternative of depth j hangs off chain row j-1: it sees rows 0..j-1 and itself.
__global__ void begin_verify_tree_kernel(DevState* st, int n, const int* __restrict__ cand, const int* __restrict__ cand_n, int budget)
{
    const int k = st->n_drafted;
    set_causal_rows(st);
    int used = k + 1;
    for (int j = 1; j <= k; ++j) {
        int extra = min(cand_n[j - 1] - 1, budget - used);
        for (int i = 1; i <= extra; ++i) {
            st->draft_tok[used] = cand[(j - 1) * TREE_TOPK + i];
            st->row_depth[used] = j;
            st->row_parent[used] = j - 1;
            st->row_vis[used] = ((1u << j) - 1u) | (1u << used);
            ++used;
        }
    }
    st->pos0 = n;
    st->n_rows = used;
    st->tok_off = 0;
    st->tree_rows = used;
}

// Verification of a tree the caller spelled out: tokens in st->draft_tok[0..rows), parents in st->row_parent (copied
// there beforehand, parent[i] < i, parent[0] = -1): fills depths and visibility.
__global__ void begin_verify_given_tree_kernel(DevState* st, int n, int rows)
{
    st->row_depth[0] = 0;
    st->row_vis[0] = 1u;
    for (int m = 1; m < rows; ++m) {
        const int p = st->row_parent[m];
        st->row_depth[m] = st->row_depth[p] + 1;
        st->row_vis[m] = st->row_vis[p] | (1u << m);
    }
    st->pos0 = n;
    st->n_rows = rows;
    st->tok_off = 0;
    st->tree_rows = rows;
    st->n_drafted = rows - 1;
}

// After a tree was accepted: the accepted node of depth j belongs in cache slot pos0 + j; one that was verified in
// another slot (an alternative) is moved there, K and V of every block.  grid = (n_blocks, 2), any block size.
template <typename T>
__global__ void kv_move_accepted_kernel(const DevState* st, T* __restrict__ kv_pool, const int* __restrict__ page_table, KvLayout L, int pos0)
{
    if (st->tree_rows == 0) return;
    const int block = blockIdx.x, kv = blockIdx.y, per = L.n_kv_heads * L.head_dim;
    for (int j = 1; j <= st->n_accepted; ++j) {                  // ascending depth: a slot is never needed after it was overwritten
        const int src = pos0 + st->acc_row[j - 1], dst = pos0 + j;
        if (src == dst) continue;
        const int ps = page_table[src >> L.page_shift], pd = page_table[dst >> L.page_shift];
        for (int i = threadIdx.x; i < per; i += blockDim.x) {
            const int h = i / L.head_dim, d = i - h * L.head_dim;
            kv_pool[L.offset(pd, block, kv, h, dst & (L.page_size - 1)) + d] = kv_pool[L.offset(ps, block, kv, h, src & (L.page_size - 1)) + d];
        }
        __syncthreads();
    }
}

// Precomputed rotary table: cs[pos][i] = (cos, sin)(pos * theta^(-2i/dh)), evaluated in double.
__global__ void rope_table_kernel(float2* cs, int max_positions, int half, double theta)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= max_positions * half) return;
    const int pos = idx / half, i = idx % half;
    const double inv_freq = pow(theta, -(double)i / (double)half);
    double s, c;
    sincos((double)pos * inv_freq, &s, &c);
    cs[idx] = make_float2((float)c, (float)s);
}

// Copies whole KV pages (all blocks) src_page -> dst_page: copy-on-write for candidate scoring.
__global__ void page_copy_kernel(uint4* pool, size_t page_vec16, int src_page, int dst_page)
{
    const uint4* s = pool + (size_t)src_page * page_vec16;
    uint4* d = pool + (size_t)dst_page * page_vec16;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < page_vec16; i += (size_t)gridDim.x * blockDim.x)
        d[i] = s[i];
}

// Gathers K or V of one block for positions [pos0, pos0+count) into fp32 [count][Hkv][dh] (inspection).
template <typename T>
__global__ void kv_read_kernel(const T* __restrict__ kv_pool, const int* __restrict__ page_table, KvLayout L, int block,
                               int which, int pos0, int count, float* __restrict__ out)
{
    const size_t total = (size_t)count * L.n_kv_heads * L.head_dim;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int d = (int)(i % L.head_dim);
        const int hk = (int)((i / L.head_dim) % L.n_kv_heads);
        const int pos = pos0 + (int)(i / ((size_t)L.head_dim * L.n_kv_heads));
        out[i] = to_float(kv_pool[L.offset(page_table[pos >> L.page_shift], block, which, hk, pos & (L.page_size - 1)) + d]);
    }
}

// ------------------------------------------------------------------------------ embedding
template <typename T>
__global__ void embed_kernel(DevState* st, const int* __restrict__ toks, const T* __restrict__ embed,
                             float* __restrict__ h, int d, int vocab)
{
    pdl_enter();
    const int r = blockIdx.x;
    if (r >= st->n_rows) return;
    int tok = toks[st->tok_off + r];
    if (tok < 0 || tok >= vocab) {
        if (threadIdx.x == 0) st->error = 1;
        tok = 0;
    }
    const T* src = embed + (size_t)tok * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)r * d + i] = to_float(src[i]);
}

// Embedding gather for the fused tensor-core walk: besides h it stores the hi/lo planes of h * gain
// (gain of the first RMSNorm that will see this row) and the row's sum of squares as "tile 0".
template <typename T>
__global__ void embed_fused_kernel(DevState* st, const int* __restrict__ toks, const T* __restrict__ embed,
                                   float* __restrict__ h, const float* __restrict__ gain, __nv_bfloat16* __restrict__ planes,
                                   float* __restrict__ sumsq_out, int d, int vocab)
{
    pdl_enter();
    __shared__ float red[33];
    const int r = blockIdx.x;
    if (r >= st->n_rows) return;
    int tok = toks[st->tok_off + r];
    if (tok < 0 || tok >= vocab) {
        if (threadIdx.x == 0) st->error = 1;
        tok = 0;
    }
    const T* src = embed + (size_t)tok * d;
    float ss = 0.f;
#pragma unroll 4
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = to_float(src[i]);
        h[(size_t)r * d + i] = v;
        if (gain) store_hi_lo(planes, r, d, i, v * gain[i]);
        ss += v * v;
    }
    const float total = block_sum(ss, red);
    if (threadIdx.x == 0) sumsq_out[r] = total;
}

// ------------------------------------------------------------------------------ residual + RMSNorm
// h[r,:] += sum_s part[s][r][:]  (the pending output of the previous residual branch, split-K
// partial sums added in split order), then x[r,:] = h * rsqrt(mean(h^2) + eps) * g.
__global__ void __launch_bounds__(512) resid_norm_kernel(const DevState* st, float* __restrict__ h,
                                                         const float* __restrict__ part, int n_split,
                                                         size_t split_stride, const float* __restrict__ gain,
                                                         float* __restrict__ x, __nv_bfloat16* __restrict__ planes,
                                                         int d, float eps)
{
    pdl_enter();
    __shared__ float red[33];
    const int r = blockIdx.x;
    if (r >= st->n_rows) return;
    float* hr = h + (size_t)r * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = hr[i];
        for (int s = 0; s < n_split; ++s) v += part[s * split_stride + (size_t)r * d + i];
        hr[i] = v;
        ss += v * v;
    }
    const float total = block_sum(ss, red);
    const float rstd = rsqrtf(total / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = hr[i] * rstd * gain[i];
        x[(size_t)r * d + i] = v;
        if (planes) store_hi_lo(planes, r, d, i, v);
    }
}

// ------------------------------------------------------------------------------ RoPE + KV append
// Sums the fused QKV projection's split-K partials, rotates q and k (rotate-half pairing: dim i
// with i + dh/2) by the row's absolute position, writes q (fp32) for the attention kernel and k, v
// into the paged cache.  grid = (rows, H + 2*Hkv), block = dh/2 threads.
template <typename T>
__global__ void qkv_post_kernel(const DevState* st, const float* __restrict__ part, int n_split, size_t split_stride,
                                int n_qkv, float* __restrict__ q_out, T* __restrict__ kv_pool,
                                const int* __restrict__ page_table, KvLayout L, int block, int n_heads,
                                const float2* __restrict__ rope_cs, int max_positions)
{
    pdl_enter();
    const int r = blockIdx.x;
    if (r >= st->n_rows) return;
    const int head = blockIdx.y, half = L.head_dim >> 1, i = threadIdx.x;
    const int pos = st->pos0 + r;                       // cache slot of the row; its sequence position follows its depth
    const int rpos = st->pos0 + st->row_depth[r];
    if (pos >= max_positions) return;
    const size_t col = (size_t)head * L.head_dim + i;
    float a = 0.f, b = 0.f;
    for (int s = 0; s < n_split; ++s) {
        const float* p = part + s * split_stride + (size_t)r * n_qkv + col;
        a += p[0];
        b += p[half];
    }
    const float2 cs = rope_cs[(size_t)rpos * half + i];
    if (head < n_heads) {
        float* q = q_out + (size_t)r * n_heads * L.head_dim + col;
        q[0] = a * cs.x - b * cs.y;
        q[half] = b * cs.x + a * cs.y;
    } else {
        const int hk = head - n_heads;
        const int kv = hk >= L.n_kv_heads ? 1 : 0;
        const int kh = kv ? hk - L.n_kv_heads : hk;
        const int page = page_table[pos >> L.page_shift];
        T* dst = kv_pool + L.offset(page, block, kv, kh, pos & (L.page_size - 1)) + i;
        if (kv == 0) {
            store_val(dst, a * cs.x - b * cs.y);
            store_val(dst + half, b * cs.x + a * cs.y);
        } else {
            store_val(dst, a);
            store_val(dst + half, b);
        }
    }
}

// ------------------------------------------------------------------------------ SwiGLU
// act[r][i] = silu(gate_i) * up_i from the fused gate/up projection, whose output columns are
// interleaved in groups of 16: [g0..g15, u0..u15, g16..g31, u16..u31, ...].
__global__ void swiglu_kernel(const DevState* st, const float* __restrict__ part, int n_split, size_t split_stride,
                              float* __restrict__ act, __nv_bfloat16* __restrict__ planes, int ffn)
{
    pdl_enter();
    const int r = blockIdx.y;
    if (r >= st->n_rows) return;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= ffn) return;
    const size_t gi = (size_t)(i >> 4) * 32 + (i & 15);
    float g = 0.f, u = 0.f;
    for (int s = 0; s < n_split; ++s) {
        const float* p = part + s * split_stride + (size_t)r * 2 * ffn;
        g += p[gi];
        u += p[gi + 16];
    }
    const float v = g / (1.f + expf(-g)) * u;
    act[(size_t)r * ffn + i] = v;
    if (planes) store_hi_lo(planes, r, ffn, i, v);
}

} // namespace swk

namespace swk {

// ------------------------------------------------------------------------------ candidate scoring, all candidates at once
// Every candidate skip set keeps its own copy of the window's residual rows in H_all[c * gamma + i]; a sub-layer is
// applied to the candidates that keep it, their rows taken in chunks of up to 128 through a row map: the norm's planes
// are gathered, the sub-layer's last GEMM adds to the residual rows in place (Eq. 2 evaluates all candidates on the same
// gamma context tokens, "Parallel Candidate Evaluation", Section 4.1).

// H_all[row] = embedding of the window token row % gamma.  grid = rows, any block size.
template <typename T>
__global__ void embed_rows_kernel(DevState* st, const int* __restrict__ toks, const T* __restrict__ embed, float* __restrict__ H_all,
                                  int d, int vocab, int gamma)
{
    const int row = blockIdx.x;
    int tok = toks[row % gamma];
    if (tok < 0 || tok >= vocab) {
        if (threadIdx.x == 0) st->error = 1;
        tok = 0;
    }
    const T* src = embed + (size_t)tok * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) H_all[(size_t)row * d + i] = to_float(src[i]);
}

// Chunk row r = H_all[rowmap[r]]: stores the hi/lo planes of that residual row * gain (the input of the sub-layer's
// first GEMM) and the row's sum of squares as "tile 0"; the residual row itself stays where it is (the sub-layer's last
// GEMM adds to it in place, through the same map).  grid = chunk rows, block = 1024.
__global__ void gather_norm_kernel(const int* __restrict__ rowmap, const float* __restrict__ H_all,
                                   const float* __restrict__ gain, __nv_bfloat16* __restrict__ planes, float* __restrict__ sumsq_out, int d)
{
    __shared__ float red[33];
    const int r = blockIdx.x;
    const float* src = H_all + (size_t)rowmap[r] * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = src[i];
        store_hi_lo(planes, r, d, i, v * gain[i]);
        ss += v * v;
    }
    const float total = block_sum(ss, red);
    if (threadIdx.x == 0) sumsq_out[r] = total;
}

// out[row] = arg max of logits[row][:], lowest token id among equals.  grid = rows, block = 1024.
__global__ void __launch_bounds__(1024) argmax_rows_kernel(const float* __restrict__ logits, int vocab, int* __restrict__ out)
{
    __shared__ float sv[32];
    __shared__ int si[32];
    const float* row = logits + (size_t)blockIdx.x * vocab;
    float bv = -INFINITY;
    int bi = 0x7FFFFFFF;
    for (int i = threadIdx.x; i < vocab; i += blockDim.x) {
        const float v = row[i];
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x < 32) {
        bv = threadIdx.x < (blockDim.x >> 5) ? sv[threadIdx.x] : -INFINITY;
        bi = threadIdx.x < (blockDim.x >> 5) ? si[threadIdx.x] : 0x7FFFFFFF;
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (threadIdx.x == 0) out[blockIdx.x] = bi;
    }
}

// counts[c] = #{ i < gamma : pred[c * gamma + i] == truth[i] } (the numerator of Eq. 3).  One thread per candidate.
__global__ void match_rows_kernel(const int* __restrict__ pred, const int* __restrict__ truth, int gamma, int n_cand, int* __restrict__ counts)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n_cand) return;
    int m = 0;
    for (int i = 0; i < gamma; ++i) m += pred[c * gamma + i] == truth[i] ? 1 : 0;
    counts[c] = m;
}

} // namespace swk
