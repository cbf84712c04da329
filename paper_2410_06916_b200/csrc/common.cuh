// Shared device-side definitions of the SWIFT hot path (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace swk {

constexpr int ROWS = 16;          // rows of one forward chunk (pending token + up to 15 drafts)
constexpr int ATTN_CHUNK = 64;    // KV positions per attention split; anchored at multiples of this
constexpr int MAX_SCORE_ROWS = 128;
constexpr int TREE_TOPK = 10;        // most predictions one draft position is extended with (Section 4.2)

// purposes of a random draw inside one decoding round (Philox counter word 2)
enum { DRAW_DRAFT = 0, DRAW_ACCEPT = 1, DRAW_RESAMPLE = 2, DRAW_BONUS = 3 };
enum { VOCAB_PLAIN = 0, VOCAB_DRAFT = 1 };

// Device-resident control block.  Every kernel of a forward reads its row count and base position
// from here, so a forward can be enqueued before the host knows how many rows it will have
// (early-stopped drafting) and replayed without new arguments.
struct DevState {
    int pos0;        // position of row 0 of the current forward
    int n_rows;      // valid rows of the current forward; 0 turns every kernel into a no-op
    int tok_off;     // offset into the token array the embedding reads
    int active;      // drafting still running
    int n_drafted;   // k: draft tokens produced in this round
    int error;       // sticky error word (bad token id, ...)
    int n_accepted;  // a
    int next_token;  // token chosen by the acceptance step
    int draft_tok[ROWS];   // [0] = pending token t*, [j] = y'_j
    float conf[ROWS];      // p_j = max softmax of draft step j (index j-1)
    int row_tok[ROWS];     // tokens of a generic forward chunk
    int argmax[ROWS];      // per-row argmax of the last forward that ran the output head
    float row_max[ROWS];   // per-row max logit
    float row_sum[ROWS];   // per-row sum exp((l - max) / T)
    int match_count;       // score_skipsets: matches of the current candidate
    int draft_j;           // index (1-based) of the draft step in flight
    int round;             // round counter = Philox counter word 0
    float stop_conf;       // early-stop threshold of this round
    unsigned seed_lo, seed_hi;
    int pad[2];
    float row_thresh[ROWS]; // nucleus sampling: smallest exp((l - max) / T) a row keeps (0 = everything); row_sum covers the kept ones
    // Shape of the forward's own rows.  Row m is stored at cache slot pos0 + m; it sits at sequence position
    // pos0 + row_depth[m] (rotary embedding) and sees row j of the forward iff bit j of row_vis[m] is set.  A plain
    // forward has depth m and bits 0..m (causal order); a verified token tree has a node's depth and its ancestors.
    unsigned row_vis[ROWS];
    int row_depth[ROWS];
    // Token tree of a verification (dynamic verification, Section 4.2): parent row of every row (-1 for row 0), and
    // after acceptance the rows of the accepted nodes in order (acc_row[j-1] = row of the accepted node of depth j).
    int row_parent[ROWS];
    int acc_row[ROWS];
    int tree_rows;         // rows of the verified tree; 0 = the verification held the drafted chain only
    int pad2[3];
};

// Causal order over the forward's rows: the default shape.
__device__ __forceinline__ void set_causal_rows(DevState* st)
{
    for (int m = 0; m < ROWS; ++m) {
        st->row_vis[m] = (2u << m) - 1u;
        st->row_depth[m] = m;
        st->row_parent[m] = m - 1;
    }
    st->tree_rows = 0;
}

// Programmatic dependent launch.  Every kernel of a forward is launched with programmatic stream
// serialisation: it may start while its predecessor is still running, so it (a) lets its own successor
// start early and (b) waits for the predecessor's completion and memory before touching anything the
// predecessor produced.  Every thread calls pdl_wait() on every path, or the chain of completions
// would be broken for the kernels that follow.  Without the launch attribute both are no-ops.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_trigger(); pdl_wait(); }

template <typename T> struct Vec;
template <> struct Vec<float> { static constexpr int N = 4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int N = 8; };

// 16-byte load of VEC elements widened to fp32
__device__ __forceinline__ void load_vec(const float* p, float (&out)[4])
{
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
__device__ __forceinline__ void load_vec(const __nv_bfloat16* p, float (&out)[8])
{
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(w[i] << 16);
        out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}
// streaming variant for weights: read once, do not keep in L1
__device__ __forceinline__ void load_vec_stream(const float* p, float (&out)[4])
{
    float4 v = __ldcs(reinterpret_cast<const float4*>(p));
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
__device__ __forceinline__ void load_vec_stream(const __nv_bfloat16* p, float (&out)[8])
{
    uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(w[i] << 16);
        out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void store_val(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_val(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// Block-wide sum; `red` is shared scratch of >= 33 floats.  All threads get the result.
__device__ __forceinline__ float block_sum(float v, float* red)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    if (w == 0) {
        float t = lane < nw ? red[lane] : 0.f;
        t = warp_sum(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    const float out = red[32];
    __syncthreads();                 // the scratch may be reused right after the call
    return out;
}

// Philox4x32-10 from its published definition (Salmon et al., SC'11).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}
// u in [0,1): top 24 bits of the first word at counter (round, slot, purpose, 0)
__device__ __forceinline__ float philox_uniform(uint64_t seed, uint32_t round, uint32_t slot, uint32_t purpose)
{
    const uint4 r = philox4x32_10(make_uint4(round, slot, purpose, 0u),
                                  make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
    return (float)(r.x >> 8) * (1.0f / 16777216.0f);
}

// Where K (kv = 0) or V (kv = 1) of (block, kv head, position) lives in the paged pool:
// pool[page][block][kv][head][slot][d].
struct KvLayout {
    int n_blocks, n_kv_heads, head_dim, page_size, page_shift;
    __device__ __forceinline__ size_t offset(int page, int block, int kv, int head, int slot) const
    {
        return ((((size_t)page * n_blocks + block) * 2 + kv) * n_kv_heads + head) * (size_t)page_size * head_dim +
               (size_t)slot * head_dim;
    }
};

} // namespace swk
