// Skinny weight-streaming GEMM on the 5th-generation tensor cores (sm_100a):
//     Y[r][n] = sum_k X[r][k] * W[n][k],   r < 16 rows,  W bf16 [N][K] streamed once from HBM.
//
// The contraction is "swapped": the 128 weight rows of a tile are the M side of tcgen05.mma, the
// rows of X are its N side.  X is fp32 upstream; it reaches the tensor cores as two bf16 planes,
// hi = bf16(x) and lo = bf16(x - hi), stacked as 32 operand rows, and the epilogue adds the two
// accumulator columns, so activations keep ~16 mantissa bits while the weights stay the only
// rounded quantity.  The kernel is HBM-bound (<= 26 flop per weight byte); tensor cores are simply
// the cheapest way to keep the arithmetic out of the way.
//
// Work decomposition (stream-K): the (tile, 64-wide k-block) units are numbered tile-major and cut
// into gridDim.x equal contiguous ranges, one per persistent CTA, so every SM streams the same
// number of bytes whatever N and K are.  A CTA whose range covers only part of a tile writes its
// partial accumulator to a slab; the last CTA to finish a tile (per-tile arrival counter) adds the
// slabs in slab order and writes Y, which makes the result independent of arrival order and of the
// row count.  A CTA that finds all the other segments of its tile already arrived skips its own slab
// and arrival and adds the others' slabs, fetched early, to its registers in the same order.
//
// What surrounds the stream matters as much as the stream at these sizes (tens of microseconds per
// launch): one weight tile is requested before the set-up barrier and the rest from the producer
// loop (a full ring from every CTA at once delayed the first tile by 3 us); per-row epilogue loops
// are rolled over the rows that exist (the last tile's epilogue runs once, from cold instruction
// caches); and once a CTA has requested all of its own tiles it asks L2 for the first tiles it
// will stream in the GEMM that follows, which fills the idle HBM time around the kernel boundary.
//
// Pipeline per CTA: warp 0 issues TMA loads (weights 128x64 + activations 32x64 per stage, 128-byte
// swizzle) into a 9-stage shared-memory ring guarded by mbarriers; warp 1 issues tcgen05.mma from
// shared memory into a double-buffered TMEM accumulator; warps 2-5 drain TMEM with tcgen05.ld, add
// the hi/lo columns and store.  Every mbarrier wait is bounded; on expiry the kernel records an
// error and winds down (TMEM is always released).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace swk {

constexpr int TC_TILE_N = 128;      // weight rows per tile (MMA M)
constexpr int TC_COLS = 32;         // operand rows of X: 16 hi + 16 lo (MMA N)
constexpr int TC_BK = 64;           // k elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int TC_STAGES = 9;        // 144 KB of weight tiles in flight per SM: HBM latency (~2 us) x 44 GB/s per SM needs ~90 KB
constexpr int TC_THREADS = 192;
constexpr int TC_A_BYTES = TC_TILE_N * TC_BK * 2;   // 16384
constexpr int TC_B_BYTES = TC_COLS * TC_BK * 2;     // 4096
constexpr int TC_PRE = 1;           // tiles requested before the set-up barrier (see the producer's comment)
constexpr int TC_STAGE_BYTES = TC_A_BYTES + TC_B_BYTES;
constexpr int TC_SMEM_BYTES = TC_STAGES * TC_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr long long TC_WAIT_CYCLES = 3000000000LL;  // ~1.5 s of SM clocks before a wait is declared dead

// The same kernel serves forwards of up to 16 rows (NB = 1: decoding) and of up to 16 * NB rows (NB = 2, 4, 8: prefill
// chunks and candidate scoring).  Rows come in blocks of 16; block rb occupies operand rows / accumulator columns
// [32 rb, 32 rb + 32): its 16 hi rows, then its 16 lo rows.  More rows per weight tile mean a wider MMA (N = 32 NB), a
// larger activation tile per stage and fewer stages in the same shared memory.  With many rows the kernel is bound by
// tensor work, not by HBM: the host then picks the grid per shape (whole tiles per CTA where a shape has enough tiles,
// tiles shared between a few CTAs where it has too few to occupy the SMs), a shared tile's partial accumulators are
// parked as the 16 values each epilogue thread holds, and the epilogue finishes one 16-row block at a time with the
// global-memory operands of the next block already requested.
template <int NB>
struct TcShape {
    static constexpr int COLS = TC_COLS * NB;                        // MMA N
    static constexpr int B_BYTES = COLS * TC_BK * 2;
    static constexpr int STAGE_BYTES = TC_A_BYTES + B_BYTES;
    static constexpr int STAGES = NB == 1 ? TC_STAGES : (196 * 1024) / STAGE_BYTES;   // 8, 6, 4 stages for NB = 2, 4, 8
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
    static constexpr int TMEM_COLS = 2 * COLS;                       // two accumulator buffers; 64 .. 512, a power of two
    static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(COLS >> 3) << 17) | ((uint32_t)(TC_TILE_N >> 4) << 24);
    static constexpr int ROWS_MAX = ROWS * NB;
};
constexpr int TC_NB_MAX = 8;
constexpr int TC_ROWS_MAX = ROWS * TC_NB_MAX;       // rows one accumulator tile covers (the wide form's "problem")
constexpr int TC_PROBS_MAX = 4;                     // problems a launch of the wide form may hold: row ranges of TC_ROWS_MAX rows that share
                                                    // the weights but nothing else; work tile T = weight tile T / n_prob of problem T % n_prob
constexpr int TC_BIG_ROWS = TC_ROWS_MAX * TC_PROBS_MAX;   // rows of the largest forward chunk
constexpr int TC_ERR_TIMEOUT = 2;

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on a phase parity.  Returns false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit_cycles = TC_WAIT_CYCLES)
{
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u && clock64() - t0 > limit_cycles) return false;
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; bf16 inputs, fp32 accumulate, M = 128, N = 32, K = 16
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes, 128-byte swizzle, groups
// of 8 rows 1024 bytes apart; descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N = 32, M = 128.
constexpr uint32_t TC_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TC_COLS >> 3) << 17) | ((uint32_t)(TC_TILE_N >> 4) << 24);

// Arrival on a counter that both publishes this CTA's earlier stores and, for the CTA that turns out to be
// last, acquires everybody else's: one acq_rel atomic at GPU scope instead of fence + atomic + fence.
// Stores of the CTA's other threads are covered through the CTA barrier that precedes it (cumulativity).
__device__ __forceinline__ int atom_add_acq_rel_gpu(int* p, int v)
{
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

// A 4-byte read whose value nobody uses: it pulls the address translation (and the line) of a location this
// thread is going to store to later, so that the store at the end of the tile does not wait for a page walk.
__device__ __forceinline__ void touch_global(const void* p)
{
    unsigned v;
    const unsigned long long a = reinterpret_cast<unsigned long long>(p) & ~3ull;   // the word that holds *p
    asm volatile("ld.global.cg.b32 %0, [%1];" : "=r"(v) : "l"(a) : "memory");
    (void)v;
}

__device__ __forceinline__ int ld_acquire_gpu(const int* p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Static stream-K schedule shared by host and device: CTA g owns units [start(g), start(g+1)).
struct StreamK {
    long long U;   // units = n_tiles * KB
    int G, KB;
    __host__ __device__ long long start(int g) const
    {
        if (U < (1ll << 31) / (G + 1)) return (long long)((unsigned)U * (unsigned)g / (unsigned)G);   // same value, 32-bit divide
        return (U * g) / G;
    }
    __host__ __device__ int owner(long long u) const      // the CTA whose range contains unit u
    {
        int g = (int)((u * G) / U);
        while (g + 1 < G && start(g + 1) <= u) ++g;
        while (g > 0 && start(g) > u) --g;
        return g;
    }
};

// fp32 rows -> the two bf16 planes the tensor-core GEMM reads, in blocks of 16 rows: row r of the forward sits in block
// r / 16; a block is 32 operand rows, hi = bf16(x) in its first 16 and lo = bf16(x - hi) in its last 16.
__device__ __forceinline__ void store_hi_lo(__nv_bfloat16* planes, int r, int K, int i, float x)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    const size_t row = (size_t)(r >> 4) * (2 * ROWS) + (r & (ROWS - 1));
    planes[row * K + i] = hi;
    planes[(row + ROWS) * K + i] = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// What the epilogue does with a finished output tile.  The element-wise steps of the decoder walk are
// folded in here so that a block of the model is four GEMM launches plus the attention pair:
//   EPI_PLAIN : Y = acc * rstd                                    (output head; rstd = 1 without a norm)
//   EPI_QKV   : acc * rstd -> RoPE on q and k -> q buffer (fp32) and K,V into the paged cache
//   EPI_SWIGLU: acc * rstd -> silu(gate) * up -> hi/lo planes of the down projection's input
//   EPI_RESID : h += acc; hi/lo planes of h * gain_next; per-tile sums of h^2 for the next RMSNorm
// RMSNorm is split around the GEMM that follows it: the producer (EPI_RESID, or the embedding gather)
// stores h * gain and the row's sum of squares in per-tile pieces; the consumer multiplies its
// accumulators by rstd = rsqrt(sum / d + eps), which is the same product in a different order.
enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_SWIGLU = 2, EPI_RESID = 3 };

struct EpiParams {
    // consumer side of the norm
    const float* sumsq_in;   // [n_sumsq_tiles][ROWS] or null (no norm in front of this GEMM)
    int n_sumsq_tiles;
    float inv_d, eps;
    // EPI_RESID
    float* h;                       // [ROWS][N] residual stream
    const int* h_rows;              // many-row form only: the 16-row block that starts at chunk row r lives in rows h_rows[r] ..
                                    // h_rows[r] + 15 of h (only multiples of 16 are looked up; null: rows r .. r + 15)
    const float* gain_next;         // [N] gain of the next RMSNorm, or null when nothing follows
    __nv_bfloat16* planes_out;      // [2*ROWS][N]
    float* sumsq_out;               // [n_tiles][ROWS]
    // EPI_SWIGLU
    __nv_bfloat16* act_planes;      // [2*ROWS][ffn]
    int ffn;
    // EPI_QKV
    float* q_out;                   // [ROWS][n_heads*dh]
    void* kv_pool;
    const int* page_table;
    KvLayout L;
    int block, n_heads, max_positions;
    const float2* rope_cs;
    int sum_rows;                   // rows per tile in sumsq_in / sumsq_out: 16 for decoding, 16 * NB for chunks of many rows
    // EPI_QKV on a chunk that holds several sequences side by side (candidate scoring: every candidate's window rows, each
    // with its own scratch pages): per 16-row block, the cache slot of its first row and the page table of its sequence
    int per_block;
    int rb_pos0[8 * TC_PROBS_MAX];
    const int* rb_page_table[8 * TC_PROBS_MAX];
    // any epilogue: shape of the GEMM that runs next on this stream (0 = none): each CTA asks for the first
    // weight tiles it will need there to be brought into L2 while this launch drains
    int next_N, next_K, next_tiles;
};

// row0: first row of the 16-row block this call finishes (0 when decoding); n_rows: rows of that block that exist;
// pos0: cache slot of row row0; rstd_sh / rope_sh / page_sh are indexed by the row within the block.
template <int EPI, typename TKV>
__device__ __forceinline__ void tc_finalize(const EpiParams& ep, int pos0, float (&val)[ROWS], int n_rows, int tile,
                                            int quarter, int lane, int etid, int N, float* Y, const float* rstd_sh,
                                            float* stage_sh, const float (&h_pre)[ROWS], float gain_pre,
                                            const float2* rope_sh, const int* page_sh, int row0 = 0)
{
    // h_pre / gain_pre (EPI_RESID) and rope_sh / page_sh (EPI_QKV) were fetched while the accumulator was still
    // being computed, so that nothing here waits for a round trip to L2 before it can store.
    const int l = quarter * 32 + lane;                 // row of the tile
    const int n = tile * TC_TILE_N + l;
    if (EPI != EPI_RESID) {
#pragma unroll
        for (int m = 0; m < ROWS; ++m) val[m] *= rstd_sh[m];
    }
    if (EPI == EPI_PLAIN) {
        if (n < N) {
#pragma unroll
            for (int m = 0; m < ROWS; ++m)
                if (m < n_rows) Y[(size_t)(row0 + m) * N + n] = val[m];
        }
    } else if (EPI == EPI_SWIGLU) {
        // rows come in groups of 32: 16 gate rows then the 16 matching up rows (same warp); staged through shared
        // memory so that the loop over the forward's rows can stay rolled
        const int i = (n >> 5) * 16 + (lane & 15);
#pragma unroll
        for (int m = 0; m < ROWS; ++m) stage_sh[m * TC_TILE_N + l] = val[m];
        __syncwarp();
        if (lane < 16 && i < ep.ffn) {
#pragma unroll 1
            for (int m = 0; m < n_rows; ++m) {
                const float g = stage_sh[m * TC_TILE_N + l], up = stage_sh[m * TC_TILE_N + l + 16];
                store_hi_lo(ep.act_planes, row0 + m, ep.ffn, i, g / (1.f + expf(-g)) * up);
            }
        }
        __syncwarp();                                  // the staging rows are rewritten by the next tile
    } else if (EPI == EPI_RESID) {
        // Rows go through shared memory so that the per-row work can be a rolled loop over the rows that exist:
        // a draft step has one, and the epilogue of the last tile is executed once, from cold instruction caches.
#pragma unroll
        for (int m = 0; m < ROWS; ++m) stage_sh[m * TC_TILE_N + l] = h_pre[m] + val[m];   // read back by this thread only
        float* sums_sh = stage_sh + ROWS * TC_TILE_N;
#pragma unroll 2                                       // two rows' shuffle chains in flight; still compact code
        for (int m = 0; m < n_rows; ++m) {
            float hn = 0.f;
            if (n < N) {
                hn = stage_sh[m * TC_TILE_N + l];
                ep.h[(size_t)(row0 + m) * N + n] = hn;
                if (ep.gain_next) store_hi_lo(ep.planes_out, row0 + m, N, n, hn * gain_pre);
            }
            if (ep.gain_next) {                        // uniform over the grid
                const float w = warp_sum(hn * hn);
                if (lane == 0) sums_sh[quarter * ROWS + m] = w;
            }
        }
        if (ep.gain_next) {
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (etid < ROWS)
                ep.sumsq_out[(size_t)tile * ep.sum_rows + row0 + etid] = etid < n_rows ?
                    (sums_sh[etid] + sums_sh[ROWS + etid]) + (sums_sh[2 * ROWS + etid] + sums_sh[3 * ROWS + etid]) : 0.f;
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
    } else {   // EPI_QKV
        // exchange through shared memory: the RoPE partner of row l sits dh/2 rows away in the same tile
#pragma unroll
        for (int m = 0; m < ROWS; ++m) stage_sh[m * TC_TILE_N + l] = val[m];
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int dh = ep.L.head_dim, half = dh >> 1;
        const int gh = n / dh, i = n - gh * dh;        // global head index (q heads, then k heads, then v heads), dim
        const int lp = i < half ? l + half : l - half;
        TKV* pool = reinterpret_cast<TKV*>(ep.kv_pool);
        if (n < N) {
#pragma unroll 1
            for (int m = 0; m < n_rows; ++m) {         // rolled on purpose: one row per draft step, and far less code to fetch
                const int pos = pos0 + m;
                if (pos < ep.max_positions) {
                    const float a = stage_sh[m * TC_TILE_N + l], b = stage_sh[m * TC_TILE_N + lp];
                    float out = a;
                    if (gh < ep.n_heads + ep.L.n_kv_heads) {      // q or k: rotate
                        const float2 cs = rope_sh[m * (TC_TILE_N / 2) + (i < half ? i : i - half)];
                        out = i < half ? a * cs.x - b * cs.y : a * cs.x + b * cs.y;
                    }
                    if (gh < ep.n_heads) {
                        ep.q_out[(size_t)(row0 + m) * ep.n_heads * dh + n] = out;
                    } else {
                        const int hk = gh - ep.n_heads;
                        const int kv = hk >= ep.L.n_kv_heads ? 1 : 0;
                        const int kh = kv ? hk - ep.L.n_kv_heads : hk;
                        store_val(pool + ep.L.offset(page_sh[m], ep.block, kv, kh, pos & (ep.L.page_size - 1)) + i, out);
                    }
                }
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");   // staging buffer is reused by the next tile
    }
}

// grid = G persistent CTAs, block = 192 threads, dynamic smem = TC_SMEM_BYTES.
// mapW: bf16 [N][K], box {64, 128}; mapX: bf16 [32][K] (rows 0-15 hi, 16-31 lo), box {64, 32}; both
// 128-byte swizzled.  slabs: [S_max][ROWS][N] fp32 (many rows: [S_max][tile][block][row of tile][16], the 16 values a
// thread holds side by side); counters: one int per tile, zero on entry and on exit.
template <int EPI, typename TKV, int NB = 1>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(DevState* st, const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapX,
               float* __restrict__ Y, float* __restrict__ slabs, int* __restrict__ counters, int N, int K,
               const __grid_constant__ EpiParams ep, const __grid_constant__ CUtensorMap mapNext, int n_prob_arg)
{
    typedef TcShape<NB> S;
    pdl_trigger();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_prob = NB > 1 ? n_prob_arg : 1;                     // problems of this launch (wide form only)
    const int n_tiles = ((N + TC_TILE_N - 1) / TC_TILE_N) * n_prob; // work tiles
    StreamK sk;
    sk.KB = (K + TC_BK - 1) / TC_BK;
    sk.U = (long long)n_tiles * sk.KB;
    sk.G = (int)(sk.U < (long long)gridDim.x ? sk.U : (long long)gridDim.x);   // never more CTAs than units: no empty ranges
    if ((int)blockIdx.x >= sk.G) { pdl_wait(); return; }
    const long long u_begin = sk.start(blockIdx.x), u_end = sk.start(blockIdx.x + 1);
    // weight rows and activation-plane rows of work tile t (the wide form: problem t % n_prob reads the plane rows of its own row range)
    auto w_row = [&](int t) { return (NB > 1 ? t / n_prob : t) * TC_TILE_N; };
    auto x_row = [&](int t) { return NB > 1 ? (t % n_prob) * S::COLS : 0; };

    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;        // swizzled tiles need 1024-byte alignment
    const uint32_t bars = base + S::STAGES * S::STAGE_BYTES;            // full[8], empty[8], tfull[2], tempty[2]
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (S::STAGES + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * S::STAGES + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * S::STAGES + 2 + b); };
    __shared__ uint32_t tmem_base_sh;
    __shared__ int last_flag_sh, peek_sh;
    __shared__ int abort_sh, epi_abort_sh;
    __shared__ float rstd_sh[ROWS * NB * (NB > 1 ? TC_PROBS_MAX : 1)];
    __shared__ float stage_sh[EPI == EPI_PLAIN ? 4 * ROWS : (NB > 1 && EPI == EPI_QKV ? 2 : 1) * ROWS * TC_TILE_N + 8 * ROWS];
    __shared__ float2 rope_sh[EPI == EPI_QKV && NB == 1 ? ROWS * (TC_TILE_N / 2) : 1];   // (cos, sin) of the rows' positions
    __shared__ int page_sh[ROWS];                                              // KV page of each row's position

    // The producer and the MMA warp need the row count before they can start; they read it here, ahead of the
    // set-up barrier, so that the trip to L2 overlaps the rest of the set-up.
    int n_rows_early = 0;
    if (tid == 0) {
        // This thread is the TMA producer.  It requests its first weight tiles right away, before the block-wide
        // set-up barrier and even before the wait for the preceding kernel (weights depend on nothing), then,
        // once that kernel's results are visible, the matching activation tiles.  Only TC_PRE tiles go out here:
        // a full ring from every CTA at once queues some 20 MB in front of each CTA's first tile, and the first
        // tile then arrives microseconds later than it does behind a short queue.
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapW) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapX) : "memory");
        for (int s = 0; s < TC_PRE; ++s) mbar_init(full_bar(s), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const int n_pre0 = (int)((u_end - u_begin) < TC_PRE ? (u_end - u_begin) : TC_PRE);
        int tile0 = (int)(u_begin / sk.KB), kb0 = (int)(u_begin - (long long)tile0 * sk.KB);
        for (int i = 0, t = tile0, k = kb0; i < n_pre0; ++i, (++k == sk.KB ? (k = 0, ++t) : 0)) {
            mbar_expect_tx(full_bar(i), S::STAGE_BYTES);
            tma_load_2d(base + i * S::STAGE_BYTES, &mapW, k * TC_BK, w_row(t), full_bar(i));
        }
        pdl_wait();
        n_rows_early = st->n_rows;
        for (int i = 0, t = tile0, k = kb0; i < n_pre0; ++i, (++k == sk.KB ? (k = 0, ++t) : 0))
            tma_load_2d(base + i * S::STAGE_BYTES + TC_A_BYTES, &mapX, k * TC_BK, x_row(t), full_bar(i));
    }
    if (warp == 1) {   // this warp sets up the remaining barriers and allocates 64 TMEM columns: two accumulator buffers of 32
        if (lane == 0) {
            for (int s = 0; s < S::STAGES; ++s) { if (s >= TC_PRE) mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
            for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
            abort_sh = 0;
            epi_abort_sh = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        pdl_wait();
        n_rows_early = st->n_rows;
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)), "r"(S::TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            const int n_pre = (int)((u_end - u_begin) < TC_PRE ? (u_end - u_begin) : TC_PRE);   // already requested above
            if (n_rows_early == 0) {                    // nothing to compute: let the requested tiles land, then leave
                for (int i = 0; i < n_pre; ++i) mbar_wait(full_bar(i), 0);
            } else {
            int it = n_pre;
            int tile = (int)((u_begin + n_pre) / sk.KB), kb = (int)((u_begin + n_pre) % sk.KB);
            for (long long u = u_begin + n_pre; u < u_end; ++u, ++it, (++kb == sk.KB ? (kb = 0, ++tile) : 0)) {
                const int s = it % S::STAGES;
                if (!mbar_wait(empty_bar(s), ((it / S::STAGES) & 1) ^ 1)) { abort_sh = 1; break; }
                const uint32_t a_dst = base + s * S::STAGE_BYTES, b_dst = a_dst + TC_A_BYTES;
                mbar_expect_tx(full_bar(s), S::STAGE_BYTES);
                tma_load_2d(a_dst, &mapW, kb * TC_BK, w_row(tile), full_bar(s));
                tma_load_2d(b_dst, &mapX, kb * TC_BK, x_row(tile), full_bar(s));
            }
            }
            if (ep.next_K > 0) {                        // everything of this launch is requested: now the next one's start
                StreamK nk;
                nk.KB = (ep.next_K + TC_BK - 1) / TC_BK;
                nk.U = (long long)((ep.next_N + TC_TILE_N - 1) / TC_TILE_N) * nk.KB;
                nk.G = (int)(nk.U < (long long)gridDim.x ? nk.U : (long long)gridDim.x);
                if ((int)blockIdx.x < nk.G) {
                    const long long u0 = nk.start(blockIdx.x), u1 = nk.start(blockIdx.x + 1);
                    int t = (int)(u0 / nk.KB), k = (int)(u0 - (long long)t * nk.KB);
                    for (int i = 0; i < ep.next_tiles && u0 + i < u1; ++i, (++k == nk.KB ? (k = 0, ++t) : 0))
                        asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];"
                                     ::"l"(&mapNext), "r"(k * TC_BK), "r"(t * TC_TILE_N) : "memory");
                }
            }
        } else {
            pdl_wait();
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        pdl_wait();
        if (lane == 0 && n_rows_early != 0) {
            int it = 0, seg = 0;
            int kb = (int)(u_begin % sk.KB);
            for (long long u = u_begin; u < u_end; ++u, ++it, (++kb == sk.KB ? (kb = 0) : 0)) {
                const bool seg_first = (u == u_begin) || kb == 0;
                const bool seg_last = (u + 1 == u_end) || kb == sk.KB - 1;
                const int buf = seg & 1;
                if (seg_first) {   // the epilogue must have drained this accumulator buffer (two segments ago)
                    if (!mbar_wait(tempty_bar(buf), ((seg >> 1) & 1) ^ 1)) { abort_sh = 1; break; }
                    tc_fence_after();
                }
                const int s = it % S::STAGES;
                if (!mbar_wait(full_bar(s), (it / S::STAGES) & 1)) { abort_sh = 1; break; }
                tc_fence_after();
                const uint32_t a_addr = base + s * S::STAGE_BYTES, b_addr = a_addr + TC_A_BYTES;
                const uint64_t a_desc = tc_smem_desc(a_addr), b_desc = tc_smem_desc(b_addr);
#pragma unroll
                for (int k = 0; k < TC_BK / 16; ++k)   // 16 bf16 = 32 bytes further along the swizzled row
                    tc_mma(tmem_base + buf * S::COLS, a_desc + 2 * k, b_desc + 2 * k, S::IDESC, (seg_first && k == 0) ? 0u : 1u);
                tc_commit(empty_bar(s));               // smem stage reusable once these MMAs have read it
                if (seg_last) { tc_commit(tfull_bar(buf)); ++seg; }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..5)
        pdl_wait();
        const int n_rows = st->n_rows;
        const int pos0_epi = st->pos0;                 // read once here rather than in every tile's epilogue
        const int quarter = warp & 3;                  // TMEM lanes this warp may read: 32*quarter ..
        const int etid = tid - 64;                     // 0..127
        int seg = 0;
        long long u = n_rows != 0 ? u_begin : u_end;
        for (int i = etid; i < ROWS * NB * n_prob; i += 128) {   // rstd of the RMSNorm in front of this GEMM (1 when there is none)
            float r = 1.f;
            if (EPI != EPI_RESID && ep.sumsq_in) {
                float ss = 0.f;
                for (int t = 0; t < ep.n_sumsq_tiles; ++t) ss += ep.sumsq_in[(size_t)t * ep.sum_rows + i];
                r = rsqrtf(ss * ep.inv_d + ep.eps);
            }
            rstd_sh[i] = r;
        }
        if (EPI == EPI_QKV && NB == 1) {
            const int half = ep.L.head_dim >> 1, pos0 = pos0_epi;
            for (int idx = etid; idx < ROWS * half; idx += 128) {
                const int m = idx / half, j = idx - m * half, pos = pos0 + m;
                // the row is stored in cache slot pos; its rotary position follows its depth (they differ in a token tree)
                if (m < n_rows && pos < ep.max_positions) rope_sh[m * (TC_TILE_N / 2) + j] = ep.rope_cs[(size_t)(pos0 + st->row_depth[m]) * half + j];
            }
            if (etid < ROWS) {
                const int pos = pos0 + etid;
                page_sh[etid] = (etid < n_rows && pos < ep.max_positions) ? ep.page_table[pos >> ep.L.page_shift] : 0;
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if constexpr (NB > 1) {
            // Chunks of many rows: the accumulator holds NB blocks of 16 rows side by side; each is drained and finished
            // (or parked in this CTA's slab) in turn.  Everything a block's finish needs from global memory (its slice
            // of the residual stream, or its rows' rotary factors and cache pages) is requested one block ahead, the
            // row loops are unrolled (this code runs NB times per tile: it is warm), and the staging buffers alternate
            // between blocks so that one barrier per block suffices.
            constexpr int RT = ROWS * NB;
            int R0 = 0;                                   // first row of the problem the current work tile belongs to
            int live_blocks = 0;                          // 16-row blocks of that problem that hold rows
            const int l = quarter * 32 + lane;
            const size_t slab_stride = (size_t)n_tiles * TC_TILE_N * RT;     // one CTA's parked partial tiles
            float* sums_sh = stage_sh + (EPI == EPI_QKV ? 2 : 1) * ROWS * TC_TILE_N;      // [2][4 * ROWS]
            struct ManyPre { float h[ROWS]; float2 cs[ROWS]; int page[ROWS]; };
            auto prefetch = [&](int rb, int n, ManyPre& p) {
                const int row0 = R0 + rb * ROWS, rows_here = min(ROWS, n_rows - row0);
                if (EPI == EPI_RESID) {
                    const float* hb = ep.h + (size_t)(ep.h_rows ? __ldg(ep.h_rows + row0) : row0) * N + n;
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) p.h[m] = (n < N && m < rows_here) ? __ldcg(hb + (size_t)m * N) : 0.f;
                } else if (EPI == EPI_QKV) {
                    const int pos_b = ep.per_block ? ep.rb_pos0[row0 / ROWS] : pos0_epi + row0;     // cache slot of the block's first row
                    const int* pt = ep.per_block ? ep.rb_page_table[row0 / ROWS] : ep.page_table;
                    const int dh = ep.L.head_dim, half = dh >> 1, i = n % dh, j = i < half ? i : i - half;
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) {
                        const int pos = pos_b + m;
                        const bool ok = m < rows_here && pos < ep.max_positions;
                        p.cs[m] = ok ? __ldg(ep.rope_cs + (size_t)pos * half + j) : make_float2(1.f, 0.f);
                        p.page[m] = ok ? __ldg(pt + (pos >> ep.L.page_shift)) : -1;
                    }
                }
            };
            auto finish_many = [&](int rb, float (&val)[ROWS], int tile, int n, const ManyPre& p, float gain) {   // tile: the weight tile
                const int row0 = R0 + rb * ROWS, rows_here = min(ROWS, n_rows - row0);
                if (EPI != EPI_RESID) {
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) val[m] *= rstd_sh[row0 + m];
                }
                if (EPI == EPI_PLAIN) {
                    if (n < N) {
#pragma unroll
                        for (int m = 0; m < ROWS; ++m)
                            if (m < rows_here) Y[(size_t)(row0 + m) * N + n] = val[m];
                    }
                } else if (EPI == EPI_SWIGLU) {
                    // lanes 0-15 hold gate rows, lanes 16-31 the matching up rows: the lower half finishes the block's
                    // rows 0-7, the upper half rows 8-15, after one exchange per row pair
                    const int i = (n >> 5) * 16 + (lane & 15);
                    const bool upper = lane >= 16;
#pragma unroll
                    for (int m = 0; m < ROWS / 2; ++m) {
                        const float recv = __shfl_xor_sync(0xffffffffu, upper ? val[m] : val[m + ROWS / 2], 16);
                        const float g = upper ? recv : val[m], up = upper ? val[m + ROWS / 2] : recv;
                        const int row = upper ? m + ROWS / 2 : m;
                        if (i < ep.ffn && row < rows_here) store_hi_lo(ep.act_planes, row0 + row, ep.ffn, i, g / (1.f + expf(-g)) * up);
                    }
                } else if (EPI == EPI_RESID) {
                    float sq[ROWS];
                    float* hb = ep.h + (size_t)(ep.h_rows ? __ldg(ep.h_rows + row0) : row0) * N + n;
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) {
                        const float hn = p.h[m] + val[m];
                        const bool ok = n < N && m < rows_here;
                        if (ok) {
                            hb[(size_t)m * N] = hn;
                            if (ep.gain_next) store_hi_lo(ep.planes_out, row0 + m, N, n, hn * gain);
                        }
                        sq[m] = ok ? hn * hn : 0.f;
                    }
                    if (ep.gain_next) {                    // uniform over the grid
                        // sums of squares per row over the warp's 32 columns: halve the rows a lane carries at every
                        // exchange; lane pair (2r, 2r + 1) ends with row r
#pragma unroll
                        for (int s = 16, len = ROWS; s >= 2; s >>= 1, len >>= 1) {
                            const bool up_half = (lane & s) != 0;
#pragma unroll
                            for (int i = 0; i < ROWS / 2; ++i)
                                if (i < len / 2) {
                                    const float keep = up_half ? sq[i + len / 2] : sq[i], send = up_half ? sq[i] : sq[i + len / 2];
                                    sq[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
                                }
                        }
                        const float tot = sq[0] + __shfl_xor_sync(0xffffffffu, sq[0], 1);
                        float* ss = sums_sh + (rb & 1) * 4 * ROWS;
                        if (!(lane & 1)) ss[quarter * ROWS + (lane >> 1)] = tot;
                        asm volatile("bar.sync 1, 128;" ::: "memory");
                        if (etid < ROWS)
                            ep.sumsq_out[(size_t)tile * ep.sum_rows + row0 + etid] = etid < rows_here ?
                                (ss[etid] + ss[ROWS + etid]) + (ss[2 * ROWS + etid] + ss[3 * ROWS + etid]) : 0.f;
                    }
                } else {   // EPI_QKV: the RoPE partner of row l sits dh/2 rows away in the same tile, in another warp
                    float* stg = stage_sh + (rb & 1) * ROWS * TC_TILE_N;
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) stg[m * TC_TILE_N + l] = val[m];
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    const int dh = ep.L.head_dim, half = dh >> 1;
                    const int gh = n / dh, i = n - gh * dh;
                    const int lp = i < half ? l + half : l - half;
                    const int pos_b = ep.per_block ? ep.rb_pos0[row0 / ROWS] : pos0_epi + row0;
                    TKV* pool = reinterpret_cast<TKV*>(ep.kv_pool);
                    const int hk = gh - ep.n_heads;
                    const int kv = hk >= ep.L.n_kv_heads ? 1 : 0;
                    const int kh = kv ? hk - ep.L.n_kv_heads : hk;
                    if (n < N) {
#pragma unroll
                        for (int m = 0; m < ROWS; ++m) {
                            if (p.page[m] >= 0) {           // the row exists and its position fits the cache
                                const float a = val[m], b = stg[m * TC_TILE_N + lp];
                                float out = a;
                                if (gh < ep.n_heads + ep.L.n_kv_heads) out = i < half ? a * p.cs[m].x - b * p.cs[m].y : a * p.cs[m].x + b * p.cs[m].y;
                                if (gh < ep.n_heads) ep.q_out[(size_t)(row0 + m) * ep.n_heads * dh + n] = out;
                                else store_val(pool + ep.L.offset(p.page[m], ep.block, kv, kh, (pos_b + m) & (ep.L.page_size - 1)) + i, out);
                            }
                        }
                    }
                }
            };
            while (u < u_end) {
                const int tile = (int)(u / sk.KB), kb0 = (int)(u % sk.KB);
                const long long tile_end = (long long)(tile + 1) * sk.KB;
                const long long seg_end = tile_end < u_end ? tile_end : u_end;
                const int buf = seg & 1;
                const int wt = tile / n_prob;              // weight tile; the problem is tile % n_prob
                R0 = (tile - wt * n_prob) * RT;
                live_blocks = (min(n_rows - R0, RT) + ROWS - 1) / ROWS;
                const int n = wt * TC_TILE_N + l;
                const bool whole = (kb0 == 0) && (seg_end == tile_end);
                int slab = 0, nseg = 1;
                if (!whole) {
                    const int g_first = sk.owner((long long)tile * sk.KB), g_last = sk.owner(tile_end - 1);
                    slab = blockIdx.x - g_first;
                    nseg = g_last - g_first + 1;
                }
                ManyPre pre;
                float gain = 0.f;
                if (whole) {
                    prefetch(0, n, pre);
                    if (EPI == EPI_RESID && ep.gain_next && n < N) gain = ep.gain_next[n];
                }
                if (!mbar_wait(tfull_bar(buf), (seg >> 1) & 1)) epi_abort_sh = 1;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (epi_abort_sh) { abort_sh = 1; break; }
                tc_fence_after();
                for (int rb = 0; rb < live_blocks; ++rb) {
                    ManyPre nxt;
                    if (whole && rb + 1 < live_blocks) prefetch(rb + 1, n, nxt);
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * S::COLS + rb * TC_COLS);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                        : "r"(taddr));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    float val[ROWS];
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) val[m] = __uint_as_float(v[m]) + __uint_as_float(v[16 + m]);
                    if (whole) {
                        finish_many(rb, val, wt, n, pre, gain);
                        pre = nxt;
                    } else {                                   // parked as this thread's 16 values side by side
                        float4* mine = reinterpret_cast<float4*>(slabs + (size_t)slab * slab_stride + (((size_t)tile * NB + rb) * TC_TILE_N + l) * ROWS);
#pragma unroll
                        for (int q4 = 0; q4 < ROWS / 4; ++q4) mine[q4] = make_float4(val[4 * q4], val[4 * q4 + 1], val[4 * q4 + 2], val[4 * q4 + 3]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(buf));   // accumulator buffer free again (4 warps arrive)
                if (!whole) {
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (etid == 0) last_flag_sh = (atom_add_acq_rel_gpu(&counters[tile], 1) == nseg - 1) ? 1 : 0;
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (last_flag_sh) {                         // last arrival: add the slabs in slab order, block by block
                        constexpr int SJ = EPI == EPI_QKV ? 2 : 3;   // slabs fetched side by side (more than that: one after another)
                        float cur[SJ][ROWS], nxs[SJ][ROWS];
                        auto fetch = [&](int rb, float (&t)[SJ][ROWS]) {
#pragma unroll
                            for (int j = 0; j < SJ; ++j) {
                                const float4* src = reinterpret_cast<const float4*>(slabs + (size_t)j * slab_stride + (((size_t)tile * NB + rb) * TC_TILE_N + l) * ROWS);
#pragma unroll
                                for (int q4 = 0; q4 < ROWS / 4; ++q4) {
                                    const float4 x = j < nseg ? __ldcg(src + q4) : make_float4(0.f, 0.f, 0.f, 0.f);
                                    t[j][4 * q4] = x.x; t[j][4 * q4 + 1] = x.y; t[j][4 * q4 + 2] = x.z; t[j][4 * q4 + 3] = x.w;
                                }
                            }
                        };
                        constexpr bool AHEAD = EPI != EPI_QKV;    // the next block's slabs are requested before this block is finished
                        if (AHEAD) fetch(0, cur);
                        prefetch(0, n, pre);
                        if (EPI == EPI_RESID && ep.gain_next && n < N) gain = ep.gain_next[n];
                        for (int rb = 0; rb < live_blocks; ++rb) {
                            ManyPre nxt;
                            if (!AHEAD) fetch(rb, cur);
                            if (rb + 1 < live_blocks) {
                                if (AHEAD) fetch(rb + 1, nxs);
                                prefetch(rb + 1, n, nxt);
                            }
                            float val[ROWS];
#pragma unroll
                            for (int m = 0; m < ROWS; ++m) val[m] = 0.f;
#pragma unroll
                            for (int j = 0; j < SJ; ++j)
                                if (j < nseg) {
#pragma unroll
                                    for (int m = 0; m < ROWS; ++m) val[m] += cur[j][m];
                                }
                            for (int j = SJ; j < nseg; ++j) {
                                const float4* src = reinterpret_cast<const float4*>(slabs + (size_t)j * slab_stride + (((size_t)tile * NB + rb) * TC_TILE_N + l) * ROWS);
#pragma unroll
                                for (int q4 = 0; q4 < ROWS / 4; ++q4) {
                                    const float4 x = __ldcg(src + q4);
                                    val[4 * q4] += x.x; val[4 * q4 + 1] += x.y; val[4 * q4 + 2] += x.z; val[4 * q4 + 3] += x.w;
                                }
                            }
                            finish_many(rb, val, wt, n, pre, gain);
                            pre = nxt;
                            if (AHEAD) {
#pragma unroll
                                for (int j = 0; j < SJ; ++j)
#pragma unroll
                                    for (int m = 0; m < ROWS; ++m) cur[j][m] = nxs[j][m];
                            }
                        }
                        if (etid == 0) counters[tile] = 0;
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                }
                ++seg;
                u = seg_end;
            }
        }
        while (NB == 1 && u < u_end) {
            const int tile = (int)(u / sk.KB), kb0 = (int)(u % sk.KB);
            const long long tile_end = (long long)(tile + 1) * sk.KB;
            const long long seg_end = tile_end < u_end ? tile_end : u_end;
            const int buf = seg & 1;
            const int n = tile * TC_TILE_N + quarter * 32 + lane;
            const bool whole = (kb0 == 0) && (seg_end == tile_end);   // this CTA covered the tile's whole K range
            // A shared tile whose other segments have all arrived already (the usual case when they sit at the start
            // of their CTAs' ranges and this one at the end of its own) needs no slab of ours and no arrival: their
            // slabs are fetched now, while the accumulator is still being computed, and added in slab order below.
            int slab = 0, nseg = 1;
            bool fast = false;
            float pre[2][ROWS];
            if (!whole) {
                const int g_first = sk.owner((long long)tile * sk.KB), g_last = sk.owner(tile_end - 1);
                slab = blockIdx.x - g_first;
                nseg = g_last - g_first + 1;
                if (etid == 0) peek_sh = ld_acquire_gpu(&counters[tile]);
                asm volatile("bar.sync 1, 128;" ::: "memory");
                fast = nseg <= 3 && peek_sh == nseg - 1;
                if (fast) {
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        const int j = jj < slab ? jj : jj + 1;          // the other segments' slabs, in slab order
#pragma unroll
                        for (int m = 0; m < ROWS; ++m)
                            pre[jj][m] = (j < nseg && n < N && m < n_rows) ? __ldcg(slabs + ((size_t)j * ROWS + m) * N + n) : 0.f;
                    }
                }
            }
            if (n < N) {                                 // where this tile's results will go (row 0 stands for all rows)
                if (EPI == EPI_PLAIN) {
                    touch_global(Y + n);
                } else if (EPI == EPI_SWIGLU) {
                    if ((n >> 5) * 16 + (lane & 15) < ep.ffn) touch_global(ep.act_planes + (n >> 5) * 16 + (lane & 15));
                } else if (EPI == EPI_RESID) {
                    if (ep.gain_next) touch_global(ep.planes_out + n);
                    if (ep.gain_next && lane == 0) touch_global(ep.sumsq_out + (size_t)tile * ep.sum_rows);
                } else {
                    const int dh = ep.L.head_dim;
                    const int gh = n / dh, i = n - gh * dh;
                    if (gh < ep.n_heads) {
                        touch_global(ep.q_out + n);
                    } else if (pos0_epi < ep.max_positions) {
                        const int hk = gh - ep.n_heads;
                        const int kv = hk >= ep.L.n_kv_heads ? 1 : 0;
                        const int kh = kv ? hk - ep.L.n_kv_heads : hk;
                        touch_global(reinterpret_cast<TKV*>(ep.kv_pool) +
                                     ep.L.offset(page_sh[0], ep.block, kv, kh, pos0_epi & (ep.L.page_size - 1)) + i);
                    }
                }
            }
            float h_pre[ROWS];
            float gain_pre = 0.f;
            if (EPI == EPI_RESID) {                     // this tile's slice of the residual stream, requested early
                const int n_pre = tile * TC_TILE_N + quarter * 32 + lane;
#pragma unroll
                for (int m = 0; m < ROWS; ++m) h_pre[m] = (n_pre < N && m < n_rows) ? __ldcg(ep.h + (size_t)m * N + n_pre) : 0.f;
                if (ep.gain_next && n_pre < N) gain_pre = ep.gain_next[n_pre];
            }
            if (!mbar_wait(tfull_bar(buf), (seg >> 1) & 1)) epi_abort_sh = 1;
            asm volatile("bar.sync 1, 128;" ::: "memory");     // all four warps agree before anyone leaves the loop
            if (epi_abort_sh) { abort_sh = 1; break; }
            tc_fence_after();
            uint32_t v[32];
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * S::COLS);
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                  "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                  "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                  "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                : "r"(taddr));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));       // accumulator buffer free again (4 warps arrive)

            float val[ROWS];
#pragma unroll
            for (int m = 0; m < ROWS; ++m) val[m] = __uint_as_float(v[m]) + __uint_as_float(v[16 + m]);
            if (whole) {
                tc_finalize<EPI, TKV>(ep, pos0_epi, val, n_rows, tile, quarter, lane, etid, N, Y, rstd_sh, stage_sh, h_pre, gain_pre, rope_sh, page_sh);
            } else if (fast) {
                // same additions as the last-arrival path below: 0 + slab 0 + slab 1 (+ slab 2), ours taken from registers
                float acc[ROWS];
#pragma unroll
                for (int m = 0; m < ROWS; ++m) {
                    const float s0 = slab == 0 ? val[m] : pre[0][m];
                    const float s1 = slab == 1 ? val[m] : (slab == 0 ? pre[0][m] : pre[1][m]);
                    float a = 0.f + s0;
                    a += s1;
                    if (nseg == 3) a += (slab == 2 ? val[m] : pre[1][m]);
                    acc[m] = a;
                }
                tc_finalize<EPI, TKV>(ep, pos0_epi, acc, n_rows, tile, quarter, lane, etid, N, Y, rstd_sh, stage_sh, h_pre, gain_pre, rope_sh, page_sh);
                if (etid == 0) counters[tile] = 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");  // peek_sh is rewritten by the next segment
            } else {
                float* mine = slabs + (size_t)slab * ROWS * N;
                if (n < N)
                    for (int m = 0; m < ROWS; ++m)
                        if (m < n_rows) mine[(size_t)m * N + n] = val[m];
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (etid == 0) last_flag_sh = (atom_add_acq_rel_gpu(&counters[tile], 1) == nseg - 1) ? 1 : 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (last_flag_sh) {                             // last arrival: add the slabs in slab order
#pragma unroll
                    for (int m = 0; m < ROWS; ++m) val[m] = 0.f;
                    if (n < N && n_rows == 1) {                 // one row: eight slabs' loads in flight at a time
                        float a = 0.f;
                        for (int j0 = 0; j0 < nseg; j0 += 8) {
                            float t8[8];
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj)
                                t8[jj] = j0 + jj < nseg ? __ldcg(slabs + (size_t)(j0 + jj) * ROWS * N + n) : 0.f;
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj)
                                if (j0 + jj < nseg) a += t8[jj];
                        }
                        val[0] = a;
                    } else if (n < N) {
                        for (int j0 = 0; j0 < nseg; j0 += 2) {      // two slabs' loads in flight at a time
#pragma unroll
                            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                                for (int m = 0; m < ROWS; ++m)
                                    pre[jj][m] = (j0 + jj < nseg && m < n_rows) ? __ldcg(slabs + ((size_t)(j0 + jj) * ROWS + m) * N + n) : 0.f;
#pragma unroll
                            for (int m = 0; m < ROWS; ++m) val[m] += pre[0][m];
                            if (j0 + 1 < nseg) {
#pragma unroll
                                for (int m = 0; m < ROWS; ++m) val[m] += pre[1][m];
                            }
                        }
                    }
                    tc_finalize<EPI, TKV>(ep, pos0_epi, val, n_rows, tile, quarter, lane, etid, N, Y, rstd_sh, stage_sh, h_pre, gain_pre, rope_sh, page_sh);
                    if (etid == 0) counters[tile] = 0;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");  // last_flag_sh and peek_sh are rewritten by the next segment
            }
            ++seg;
            u = seg_end;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (abort_sh && tid == 0) st->error = TC_ERR_TIMEOUT;
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(S::TMEM_COLS));
    }
}

// What happens when a bounded wait runs out, in its harmless form: one thread waits, with the given limit, on a barrier
// nothing ever arrives on; the wait gives up, and the kernel reports it the way the GEMM does (the error word of the
// control block) and returns normally.  No fault, no trap: the context stays usable.
__global__ void wait_probe_kernel(DevState* st, long long limit_cycles)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    if (threadIdx.x == 0) {
        const uint32_t bar = smem_u32(&bar_storage);
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(bar, 0, limit_cycles)) st->error = TC_ERR_TIMEOUT;
    }
}

// grid = (ceil(K/256), rows): splits fp32 rows [rows][K] into the planes (used when a caller supplies X directly)
// row0: row of the planes that x's first row goes to
__global__ void split_planes_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ planes, int K, int row0)
{
    const int r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < K) store_hi_lo(planes, row0 + r, K, i, x[(size_t)r * K + i]);
}

// Deterministic non-trivial contents for operand planes that a timing run would otherwise read as they happen to be
// (zeros toggle no bits in the tensor pipe and understate its power draw): values in [-0.5, 0.5), lo planes included.
__global__ void fill_planes_kernel(__nv_bfloat16* __restrict__ planes, size_t n)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        unsigned h = (unsigned)i * 2654435761u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        planes[i] = __float2bfloat16_rn((float)(h & 0xFFFF) * (1.0f / 65536.0f) - 0.5f);
    }
}

} // namespace swk
