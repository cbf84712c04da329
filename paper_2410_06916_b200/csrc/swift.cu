// Host side of the SWIFT hot-path library: context, buffer carving, the sub-layer walk that
// enqueues the kernels of one forward chunk, and the extern "C" entry points of include/swift.h.
#include "../../include/swift.h"

#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <map>
#include <tuple>
#include <mutex>
#include <vector>

#include "common.cuh"
#include "layer_opt.h"
#include "kernels_attn.cuh"
#include "kernels_attn_mma.cuh"
#include "kernels_attn_tile.cuh"
#include "kernels_elem.cuh"
#include "kernels_gemm_simt.cuh"
#include "kernels_gemm_tc.cuh"
#include "kernels_vocab.cuh"

using namespace swk;

namespace {

thread_local std::string g_load_error;

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t v, size_t a = ALIGN) { return (v + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

enum Phase { PH_LOADED = 0, PH_READY = 1, PH_DRAFTED = 2, PH_VERIFIED = 3 };

struct GemmPlan { int S, Kc; };

struct Carve {
    size_t off = 0;
    size_t take(size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; }
};

// Offsets (bytes) of every tensor inside the weights buffer.
struct WeightLayout {
    size_t embed, lm_head, final_norm, total;
    std::vector<size_t> wqkv, wo, wgu, wdown, attn_norm, mlp_norm;
};

struct WorkLayout {
    size_t state, h, xn, xa, act, q, part, o_part, ml_part, logits, q_rows, rope, pt_main, pt_score, score_tok, cand, cand_n, big_tok, score_H, score_logits, score_pred, score_maps, pt_slots,
        score_truth, score_out, attn_counters, xn_hl, xa_hl, act_hl, slabs, counters, sumsq, total;
    size_t part_floats, slab_floats;
};

struct FwdGraph;

} // namespace

struct swift_ctx {
    swift_model_desc d;
    cudaStream_t stream;
    int device;
    size_t esize;
    char* wbase; char* kvbase; char* ws;
    WeightLayout wl;
    WorkLayout kl;
    KvLayout kv;
    int n_pages_main, n_pages_scratch, max_splits;
    // host-side state
    int phase, n, pending, n_prompt, round, last_k, last_max_k;
    bool round_open;
    std::vector<int> hist;           // prompt + generated tokens, pending included
    int mode; float temperature, top_p; uint64_t seed; bool greedy_draft;
    swopt::LayerOpt* engine;         // proposal engine of swift_generate's own optimisation, kept across calls
    int tree_rows;                   // dynamic verification: rows one verification may hold (0 = off)
    DevState last_state;             // control block as last read back
    int64_t launches, h2d_bytes, d2h_bytes;
    std::string err;
    cudaEvent_t ev[8];
    // captured forwards; programmatic dependent launch between the kernels of a forward
    bool use_graphs, use_pdl, pdl_next, pdl_gemms, fuse, fuse_combine, prefetch_next, attn_mma, big_chunks, batched_scoring, whole_tiles, attn_tile, attn_tile_decode, attn_tile_drafts;
    int many_problems;              // 128-row problems per many-row GEMM launch (chunks of prefill and of candidate scoring hold that many)
    bool tree_forward = false;      // the forward being enqueued verifies a token tree (rows see their ancestors, not all earlier rows)
    int attn_rows_per_cta, prefetch_tiles;
    std::vector<FwdGraph>* graphs;
    uint64_t graph_clock;
    // per-round record of the last swift_generate (swift_round_times)
    struct RoundTime { float ms_draft, ms_verify; double bytes_draft, bytes_verify; int32_t drafted; double stored_draft, stored_verify; };
    std::vector<RoundTime> round_times;
    std::vector<uint8_t> last_mask;          // skip set in use when the last swift_generate ended (swift_final_skip_mask)
    // tensor-core GEMM path (bf16 models)
    bool use_tc;
    std::vector<CUtensorMap> tm_wqkv, tm_wo, tm_wgu, tm_wdown;
    CUtensorMap tm_lm_head, tm_embed, tm_xn, tm_xa, tm_act;
    CUtensorMap tm_xn_big, tm_xa_big, tm_act_big;      // the same planes seen as 2 * TC_BIG_ROWS operand rows, boxes of 2 * TC_ROWS_MAX (chunks of many rows)
};

namespace {

swift_status fail(swift_ctx* c, swift_status s, const char* fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (c) c->err = buf; else g_load_error = buf;
    return s;
}

// Host <-> device copy on the context's stream, counted: the totals are what a whole swift_generate call moved.
cudaError_t copy_async(swift_ctx* c, void* dst, const void* src, size_t bytes, cudaMemcpyKind kind)
{
    (kind == cudaMemcpyHostToDevice ? c->h2d_bytes : c->d2h_bytes) += (int64_t)bytes;
    return cudaMemcpyAsync(dst, src, bytes, kind, c->stream);
}

#define CU(call)                                                                                   \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess)                                                                     \
            return fail(ctx, SWIFT_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_),  \
                        __FILE__, __LINE__);                                                       \
    } while (0)

bool desc_ok(const swift_model_desc* d, std::string* why)
{
    auto bad = [&](const char* m) { if (why) *why = m; return false; };
    if (!d) return bad("null desc");
    if (d->n_blocks < 1 || d->d_model < 8 || d->n_heads < 1 || d->n_kv_heads < 1 || d->ffn < 16 || d->vocab < 2)
        return bad("non-positive dimension");
    if (d->dtype != SWIFT_F32 && d->dtype != SWIFT_BF16) return bad("dtype must be SWIFT_F32 or SWIFT_BF16");
    if (d->kv_dtype != SWIFT_F32 && d->kv_dtype != SWIFT_BF16) return bad("kv_dtype must be SWIFT_F32 or SWIFT_BF16");
    if (d->dtype == SWIFT_F32 && d->kv_dtype != SWIFT_F32) return bad("fp32 models keep an fp32 KV cache");
    if (d->n_heads % d->n_kv_heads) return bad("n_heads must be a multiple of n_kv_heads");
    if (d->head_dim < 16 || d->head_dim > 256 || (d->head_dim & (d->head_dim - 1)))
        return bad("head_dim must be a power of two in 16..256");
    if (d->d_model % 8 || d->ffn % 16 || (d->n_heads * d->head_dim) % 8) return bad("d_model%8, ffn%16 required");
    if (d->page_size < 8 || d->page_size > 128 || (d->page_size & (d->page_size - 1)))
        return bad("page_size must be a power of two in 8..128");
    if (d->max_positions < d->page_size || d->max_positions % d->page_size) return bad("max_positions must be a positive multiple of page_size");
    if (d->max_positions > 262144) return bad("max_positions is limited to 262144 (the split-combine step keeps one weight per 64 positions in shared memory)");
    if (d->max_draft < 0 || d->max_draft > SWIFT_MAX_ROWS - 1) return bad("max_draft must be in 0..15");
    if (!(d->rope_theta > 1.f) || !(d->rms_eps >= 0.f)) return bad("rope_theta > 1 and rms_eps >= 0 required");
    return true;
}

size_t esize_of(const swift_model_desc* d) { return d->dtype == SWIFT_BF16 ? 2 : 4; }
size_t kv_esize_of(const swift_model_desc* d) { return d->kv_dtype == SWIFT_BF16 ? 2 : 4; }

GemmPlan plan_gemm(const swift_model_desc* d, int N, int K)
{
    const int vec = d->dtype == SWIFT_BF16 ? 8 : 4;
    const int kc_max = 1024;                                // 16 rows x 1024 fp32 = 64 KB of shared memory
    const int gran = 32 * vec;
    const int tiles = ceil_div(N, GEMM_SIMT_TILE_N);
    int S = ceil_div(K, kc_max);
    const int want = ceil_div(2 * 148, tiles);              // at least two CTAs per SM in flight
    const int s_cap = std::max(1, K / (2 * gran));
    S = std::max(S, std::min(want, s_cap));
    int Kc = ceil_div(ceil_div(K, S), gran) * gran;
    S = ceil_div(K, Kc);
    return {S, Kc};
}

WeightLayout weight_layout(const swift_model_desc* d)
{
    WeightLayout w;
    Carve c;
    const size_t es = esize_of(d);
    const size_t dm = d->d_model, qd = (size_t)d->n_heads * d->head_dim, kd = (size_t)d->n_kv_heads * d->head_dim;
    w.embed = c.take((size_t)d->vocab * dm * es);
    for (int b = 0; b < d->n_blocks; ++b) {
        w.wqkv.push_back(c.take((qd + 2 * kd) * dm * es));
        w.wo.push_back(c.take(dm * qd * es));
        w.wgu.push_back(c.take(2 * (size_t)d->ffn * dm * es));
        w.wdown.push_back(c.take(dm * (size_t)d->ffn * es));
    }
    w.lm_head = c.take((size_t)d->vocab * dm * es);
    for (int b = 0; b < d->n_blocks; ++b) {
        w.attn_norm.push_back(c.take(dm * 4));
        w.mlp_norm.push_back(c.take(dm * 4));
    }
    w.final_norm = c.take(dm * 4);
    w.total = c.off;
    return w;
}

constexpr int TC_GRID = 148;        // persistent CTAs of the tensor-core GEMM: one per SM of a B200
constexpr int TC_MAX_TILES = 2048;       // work tiles of one launch (70B gate/up: 448 weight tiles x 4 problems)

// Largest number of CTAs that share one output tile under the stream-K schedule (= slabs needed).
int max_segments(int N, int K, int grid = TC_GRID, int n_prob = 1)
{
    StreamK sk;
    sk.KB = ceil_div(K, TC_BK);
    const int tiles = ceil_div(N, TC_TILE_N) * n_prob;      // work tiles
    sk.U = (long long)tiles * sk.KB;
    sk.G = (int)std::min<long long>(grid, sk.U);
    int worst = 1;
    for (int t = 0; t < tiles; ++t)
        worst = std::max(worst, sk.owner((long long)(t + 1) * sk.KB - 1) - sk.owner((long long)t * sk.KB) + 1);
    return worst;
}

// Grid of a many-row GEMM launch.  Such a launch is bound by tensor work, and a tile that is shared between CTAs costs
// each of them a 64 KB slab to write and the last one the others' slabs to add, so the stream-K cut is chosen per shape:
// among the grids that the slabs were sized for, the one whose busiest CTA has the least to do, counting a shared
// segment as PART_COST extra K steps and the final merge as MERGE_COST.  (40 tiles of a long K: 120 CTAs, three to a
// tile; 120 tiles: one each; 216 tiles: 144 CTAs, three tiles to a pair.)
int many_row_grid(int N, int K, int n_prob = 1)
{
    static const int forced = getenv("SWIFT_MANY_GRID") ? atoi(getenv("SWIFT_MANY_GRID")) : 0;
    constexpr long long PART_COST = 10, MERGE_COST = 14;
    static std::mutex mu;
    static std::map<std::tuple<int, int, int>, int> memo;   // the search below is far too slow for a launch path
    std::lock_guard<std::mutex> lock(mu);
    const std::tuple<int, int, int> key{N, K, n_prob};
    auto it = memo.find(key);
    if (it != memo.end()) return it->second;
    const int tiles = ceil_div(N, TC_TILE_N) * n_prob, cap = max_segments(N, K, TC_GRID, n_prob);
    if (forced > 0 && forced <= TC_GRID && max_segments(N, K, forced, n_prob) <= cap) return memo[key] = forced;
    StreamK sk;
    sk.KB = ceil_div(K, TC_BK);
    sk.U = (long long)tiles * sk.KB;
    int best = TC_GRID;
    long long best_cost = -1;
    for (int G = TC_GRID; G >= TC_GRID / 2; --G) {
        sk.G = (int)std::min<long long>(G, sk.U);
        if (max_segments(N, K, G, n_prob) > cap) continue;
        long long worst = 0;
        bool shared = false;
        for (int g = 0; g < sk.G; ++g) {
            const long long u0 = sk.start(g), u1 = sk.start(g + 1);
            long long cost = u1 - u0;
            if (u0 % sk.KB) { cost += PART_COST; shared = true; }
            if (u1 % sk.KB && (u1 / sk.KB != u0 / sk.KB || !(u0 % sk.KB))) { cost += PART_COST; shared = true; }
            worst = std::max(worst, cost);
        }
        if (shared) worst += MERGE_COST;
        if (best_cost < 0 || worst < best_cost) { best_cost = worst; best = G; }
    }
    return memo[key] = best;
}

// Scratch KV pages beyond the sequence's own: the window of one candidate (copy-on-write start page included), or the
// windows of the several candidates of one chunk when candidates are scored side by side.
int scratch_pages(const swift_model_desc* d) { return TC_PROBS_MAX * (MAX_SCORE_ROWS / d->page_size + 8); }

size_t page_bytes(const swift_model_desc* d)
{
    return (size_t)d->n_blocks * 2 * d->n_kv_heads * d->page_size * d->head_dim * kv_esize_of(d);
}

constexpr int SCORE_ROWS_MAX = 4096;     // candidates x window rows scored side by side (beyond that: one candidate at a time)
constexpr int SCORE_SLOTS_MAX = TC_BIG_ROWS / ROWS;       // candidates per chunk of TC_BIG_ROWS rows (window of 16 rows)
// Row-map entries of one scoring round: one map of a chunk's rows (128 or 256) per (sub-layer or output head, chunk of candidates).
size_t score_map_ints(const swift_model_desc* d)
{
    return (size_t)(2 * d->n_blocks + 1) * (SCORE_ROWS_MAX / TC_ROWS_MAX + SCORE_ROWS_MAX / ROWS / 2) * TC_BIG_ROWS;
}

// Rows of the largest forward chunk: TC_BIG_ROWS where the tensor-core walk with many-row chunks applies, else 16.
size_t big_rows_of(const swift_model_desc* d) { return (d->dtype == SWIFT_BF16 && d->head_dim == 128) ? (size_t)TC_BIG_ROWS : (size_t)ROWS; }

WorkLayout work_layout(const swift_model_desc* d)
{
    WorkLayout k;
    Carve c;
    const size_t es = esize_of(d);
    const size_t dm = d->d_model, qd = (size_t)d->n_heads * d->head_dim, kd = (size_t)d->n_kv_heads * d->head_dim;
    const int max_splits = ceil_div(d->max_positions, ATTN_CHUNK);
    size_t pf = 0;
    auto need = [&](int N, int K) { pf = std::max(pf, (size_t)plan_gemm(d, N, K).S * ROWS * (size_t)N); };
    need((int)(qd + 2 * kd), (int)dm); need((int)dm, (int)qd); need(2 * d->ffn, (int)dm); need((int)dm, d->ffn);
    need(d->vocab, (int)dm);
    k.part_floats = pf;
    // bf16 models with head size 128 also run chunks of up to TC_ROWS_MAX rows (prefill): their row buffers are that tall
    const size_t RB = big_rows_of(d);
    k.state = c.take(sizeof(DevState));
    k.h = c.take(RB * dm * 4);
    k.xn = c.take(ROWS * dm * 4);
    k.xa = c.take(RB * qd * 4);
    k.act = c.take(ROWS * (size_t)d->ffn * 4);
    k.q = c.take(RB * qd * 4);
    k.part = c.take(pf * 4);
    k.o_part = c.take((size_t)d->n_heads * max_splits * RB * d->head_dim * 4);
    k.ml_part = c.take((size_t)d->n_heads * max_splits * RB * 8);
    k.big_tok = c.take(RB * 4);
    // candidate scoring with all candidates side by side (chunks of many rows only): every candidate's window rows, one
    // chunk of logits, the predictions, the row maps of a whole scoring round, one page table per candidate of a chunk
    k.score_H = k.score_logits = k.score_pred = k.score_maps = k.pt_slots = 0;
    if (RB > ROWS) {
        k.score_H = c.take((size_t)SCORE_ROWS_MAX * dm * 4);
        k.score_logits = c.take(RB * (size_t)d->vocab * 4);
        k.score_pred = c.take((size_t)SCORE_ROWS_MAX * 4);
        k.score_maps = c.take(score_map_ints(d) * 4);
        k.pt_slots = c.take((size_t)SCORE_SLOTS_MAX * (d->max_positions / d->page_size) * 4);
    }
    k.logits = c.take((size_t)ROWS * d->vocab * 4);
    k.q_rows = c.take((size_t)std::max(1, d->max_draft) * d->vocab * 4);
    k.rope = c.take((size_t)d->max_positions * (d->head_dim / 2) * 8);
    const int np = d->max_positions / d->page_size;
    k.pt_main = c.take((size_t)np * 4);
    k.pt_score = c.take((size_t)np * 4);
    k.score_tok = c.take(MAX_SCORE_ROWS * 4);
    k.score_truth = c.take(MAX_SCORE_ROWS * 4);
    k.score_out = c.take(1024 * 4);
    k.cand = c.take((size_t)ROWS * TREE_TOPK * 4);
    k.cand_n = c.take(ROWS * 4);
    k.attn_counters = c.take((size_t)d->n_heads * 4);
    // tensor-core path (bf16 models): hi/lo bf16 planes of the GEMM inputs, stream-K slabs, tile counters
    k.slab_floats = 0;
    k.xn_hl = k.xa_hl = k.act_hl = k.slabs = k.counters = k.sumsq = 0;
    if (d->dtype == SWIFT_BF16) {
        auto slab_need = [&](int N, int K) {      // whole tiles: the many-row form parks 128 x RB values per tile
            int segs = max_segments(N, K);
            for (int np = 2; np <= TC_PROBS_MAX; ++np) segs = std::max(segs, max_segments(N, K, TC_GRID, np));
            k.slab_floats = std::max(k.slab_floats, (size_t)segs * RB * (size_t)ceil_div(N, TC_TILE_N) * TC_TILE_N);
        };
        slab_need((int)(qd + 2 * kd), (int)dm); slab_need((int)dm, (int)qd); slab_need(2 * d->ffn, (int)dm);
        slab_need((int)dm, d->ffn); slab_need(d->vocab, (int)dm);
        k.xn_hl = c.take(2 * RB * dm * 2);
        k.xa_hl = c.take(2 * RB * qd * 2);
        k.act_hl = c.take(2 * RB * (size_t)d->ffn * 2);
        k.slabs = c.take(k.slab_floats * 4);
        k.counters = c.take(TC_MAX_TILES * 4);
        k.sumsq = c.take((size_t)std::max(1, ceil_div((int)dm, TC_TILE_N)) * RB * 4);
    }
    k.total = c.off;
    return k;
}

template <typename T> T* wptr(swift_ctx* c, size_t off) { return reinterpret_cast<T*>(c->wbase + off); }
template <typename T> T* kptr(swift_ctx* c, size_t off) { return reinterpret_cast<T*>(c->ws + off); }
DevState* state_of(swift_ctx* c) { return kptr<DevState>(c, c->kl.state); }

int mr_of(int rows) { return rows <= 1 ? 1 : rows <= 2 ? 2 : rows <= 4 ? 4 : rows <= 8 ? 8 : 16; }
int attn_mr_of(int rows) { return rows > 8 && rows <= 12 ? 12 : mr_of(rows); }   // 9 rows = a verification of 8 drafts

// What the vocabulary kernel does on a draft row: 0 argmax (greedy mode), 1 draw from q, 2 argmax with q the point mass.
int sampling_flag(const swift_ctx* ctx) { return ctx->mode == SWIFT_SAMPLING ? (ctx->greedy_draft ? 2 : 1) : 0; }

// Dynamic shared memory of the vocabulary kernel: one float per token while a nucleus cut is searched (sampling with
// top_p < 1), if the vocabulary fits; nothing otherwise.
constexpr size_t VOCAB_CACHE_MAX_BYTES = 200 * 1024;
size_t vocab_cache_bytes(const swift_ctx* ctx)
{
    const size_t need = (size_t)ctx->d.vocab * sizeof(float);
    return (ctx->mode == SWIFT_SAMPLING && ctx->top_p < 1.f && need <= VOCAB_CACHE_MAX_BYTES) ? need : 0;
}

// ------------------------------------------------------------------------------ launches
// Launch with programmatic stream serialisation (see pdl_enter in common.cuh).
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, swift_ctx* ctx, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (ctx->use_pdl || ctx->pdl_next) ? 1 : 0;
    ctx->pdl_next = false;
    ctx->launches++;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename T, int MR>
swift_status launch_gemm_mr(swift_ctx* ctx, const float* X, int ldx, const T* W, int N, int K, GemmPlan p)
{
    const size_t smem = (size_t)MR * p.Kc * sizeof(float);
    dim3 grid(ceil_div(N, GEMM_SIMT_TILE_N), p.S);
    CU(launch_k(gemm_simt_kernel<T, MR>, grid, dim3(GEMM_SIMT_THREADS), smem, ctx, (const DevState*)state_of(ctx), X, ldx, W,
                kptr<float>(ctx, ctx->kl.part), N, K, p.Kc));
    return SWIFT_OK;
}

template <typename T>
swift_status launch_gemm(swift_ctx* ctx, int mr, const float* X, int ldx, const T* W, int N, int K, GemmPlan* plan_out)
{
    const GemmPlan p = plan_gemm(&ctx->d, N, K);
    *plan_out = p;
    switch (mr) {
    case 1: return launch_gemm_mr<T, 1>(ctx, X, ldx, W, N, K, p);
    case 2: return launch_gemm_mr<T, 2>(ctx, X, ldx, W, N, K, p);
    case 4: return launch_gemm_mr<T, 4>(ctx, X, ldx, W, N, K, p);
    case 8: return launch_gemm_mr<T, 8>(ctx, X, ldx, W, N, K, p);
    default: return launch_gemm_mr<T, 16>(ctx, X, ldx, W, N, K, p);
    }
}

// One GEMM of the walk: where its fp32 input lives, its hi/lo planes and tensor maps (tensor-core path).
struct GemmSite {
    const float* X;
    int N, K;
    const void* W;
    const CUtensorMap* mapW;
    const CUtensorMap* mapX;
};

template <int EPI, typename TKV, int NB = 1>
swift_status launch_gemm_tc(swift_ctx* ctx, const GemmSite& g, const EpiParams& ep, const CUtensorMap* next_map = nullptr, int n_prob = 1)
{
    if (ceil_div(g.N, TC_TILE_N) * n_prob > TC_MAX_TILES) return fail(ctx, SWIFT_EUNSUPPORTED, "GEMM with %d output tiles", ceil_div(g.N, TC_TILE_N) * n_prob);
    if (ctx->pdl_gemms) ctx->pdl_next = true;     // this launch may begin before its predecessor has finished (see swift_load)
    // Decoding streams each weight once and wants every SM to stream the same bytes: 148 CTAs, tiles cut where the ranges
    // fall.  A chunk of many rows is bound by its tensor work and its epilogues: see many_row_grid.
    int grid = TC_GRID;
    if (NB > 1 && ctx->whole_tiles) grid = many_row_grid(g.N, g.K, n_prob);
    CU(launch_k(gemm_tc_kernel<EPI, TKV, NB>, dim3(grid), dim3(TC_THREADS), (size_t)TcShape<NB>::SMEM_BYTES, ctx, state_of(ctx), *g.mapW, *g.mapX,
                kptr<float>(ctx, ctx->kl.part), kptr<float>(ctx, ctx->kl.slabs), kptr<int>(ctx, ctx->kl.counters), g.N, g.K, ep,
                next_map ? *next_map : *g.mapW, n_prob));
    return SWIFT_OK;
}

// The plain-epilogue GEMM of a chunk of many rows with its output at Y ([rows][N]).
template <int NB>
swift_status launch_gemm_tc_y(swift_ctx* ctx, const GemmSite& g, const EpiParams& ep, float* Y, int n_prob = 1)
{
    if (ceil_div(g.N, TC_TILE_N) * n_prob > TC_MAX_TILES) return fail(ctx, SWIFT_EUNSUPPORTED, "GEMM with %d output tiles", ceil_div(g.N, TC_TILE_N) * n_prob);
    int grid = TC_GRID;
    if (ctx->whole_tiles) grid = many_row_grid(g.N, g.K, n_prob);
    CU(launch_k(gemm_tc_kernel<EPI_PLAIN, float, NB>, dim3(grid), dim3(TC_THREADS), (size_t)TcShape<NB>::SMEM_BYTES, ctx, state_of(ctx), *g.mapW,
                *g.mapX, Y, kptr<float>(ctx, ctx->kl.slabs), kptr<int>(ctx, ctx->kl.counters), g.N, g.K, ep, *g.mapW, n_prob));
    return SWIFT_OK;
}

// Runs one GEMM site; the result lands in the `part` buffer as *n_split slabs of [ROWS][N] to be summed.
template <typename T>
swift_status run_gemm(swift_ctx* ctx, int mr, const GemmSite& g, int* n_split)
{
    if (ctx->use_tc) {
        *n_split = 1;
        EpiParams ep;
        memset(&ep, 0, sizeof ep);
        ep.sum_rows = ROWS;
        return launch_gemm_tc<EPI_PLAIN, float>(ctx, g, ep);
    }
    GemmPlan p;
    swift_status s = launch_gemm<T>(ctx, mr, g.X, g.K, reinterpret_cast<const T*>(g.W), g.N, g.K, &p);
    *n_split = p.S;
    return s;
}

template <typename T, int MR>
swift_status launch_attn_mr(swift_ctx* ctx, const int* page_table, int block, int groups, float* fused_out, __nv_bfloat16* fused_planes)
{
    const swift_model_desc& d = ctx->d;
    const size_t smem = 2 * (size_t)ATTN_CHUNK * d.head_dim * sizeof(T) + ((size_t)MR * d.head_dim + 3 * (size_t)MR * ATTN_CHUNK) * sizeof(float);
    dim3 grid(d.n_heads, ctx->max_splits);
    if (d.head_dim == 128) {
        grid.z = groups;
        const bool fused = MR == 1 && fused_out != nullptr;       // one-row forwards merge the chunks in the same launch
        CU(launch_k(attn_stream_kernel<T, MR>, grid, dim3(ATTN_THREADS), fused ? 2 * (size_t)ctx->max_splits * sizeof(float) : 0, ctx,
                    (const DevState*)state_of(ctx), (const float*)kptr<float>(ctx, ctx->kl.q), reinterpret_cast<const T*>(ctx->kvbase),
                    page_table, ctx->kv, block, d.n_heads, ctx->max_splits, 1.0f / sqrtf((float)d.head_dim),
                    kptr<float>(ctx, ctx->kl.o_part), kptr<float2>(ctx, ctx->kl.ml_part),
                    fused ? kptr<int>(ctx, ctx->kl.attn_counters) : (int*)nullptr, fused_out, fused_planes));
        return SWIFT_OK;
    }
    CU(launch_k(attn_split_kernel<T, MR>, grid, dim3(ATTN_THREADS), smem, ctx, (const DevState*)state_of(ctx),
                (const float*)kptr<float>(ctx, ctx->kl.q), reinterpret_cast<const T*>(ctx->kvbase), page_table, ctx->kv, block,
                d.n_heads, ctx->max_splits, 1.0f / sqrtf((float)d.head_dim), kptr<float>(ctx, ctx->kl.o_part),
                kptr<float2>(ctx, ctx->kl.ml_part)));
    return SWIFT_OK;
}

#define ST(call)                                   \
    do {                                           \
        swift_status s_ = (call);                  \
        if (s_ != SWIFT_OK) return s_;             \
    } while (0)

// Attention of a chunk of many rows (or of one sequence inside it): tiles of 64 query rows against 64-position chunks.
template <typename T>
swift_status launch_attn_tile(swift_ctx* ctx, const int* page_table, int block, int rows, int part_rows, int row_base, int n_rows_fixed,
                              int pos0_fixed, int n_seq = 1, int pt_stride = 0)
{
    const swift_model_desc& d = ctx->d;
    const int G = d.n_heads / d.n_kv_heads;
    // a CTA takes up to AT_TPC query tiles on one staged chunk; with several sequences the chunks that reach into their own
    // rows take one tile per CTA and sequence
    const int z = n_seq > 1 ? std::max(ceil_div(ceil_div(G * rows * n_seq, AT_QROWS), AT_TPC), n_seq * ceil_div(G * rows, AT_QROWS))
                            : ceil_div(ceil_div(G * rows, AT_QROWS), AT_TPC);
    CU(launch_k(attn_tile_kernel<T>, dim3(d.n_kv_heads, ctx->max_splits, z), dim3(AT_THREADS), AT_SMEM_BYTES, ctx,
                (const DevState*)state_of(ctx), (const float*)kptr<float>(ctx, ctx->kl.q), reinterpret_cast<const T*>(ctx->kvbase),
                page_table, ctx->kv, block, d.n_heads, ctx->max_splits, 1.0f / sqrtf((float)d.head_dim),
                kptr<float>(ctx, ctx->kl.o_part), kptr<float2>(ctx, ctx->kl.ml_part), part_rows, row_base, n_rows_fixed, pos0_fixed, n_seq,
                pt_stride));
    return SWIFT_OK;
}

template <typename T, int NT>
swift_status launch_attn_mma(swift_ctx* ctx, const int* page_table, int block, bool fused, float* out, __nv_bfloat16* planes,
                             int part_rows = ROWS, int row_base = 0, int n_rows_fixed = 0, int pos0_fixed = 0, int z_passes = 1)
{
    const swift_model_desc& d = ctx->d;
    CU(launch_k(attn_mma_kernel<T, NT>, dim3(d.n_kv_heads, ctx->max_splits, z_passes), dim3(AM_THREADS), attn_mma_smem_bytes(NT, ctx->max_splits), ctx,
                (const DevState*)state_of(ctx), (const float*)kptr<float>(ctx, ctx->kl.q), reinterpret_cast<const T*>(ctx->kvbase),
                page_table, ctx->kv, block, d.n_heads, ctx->max_splits, 1.0f / sqrtf((float)d.head_dim),
                kptr<float>(ctx, ctx->kl.o_part), kptr<float2>(ctx, ctx->kl.ml_part), part_rows,
                fused ? kptr<int>(ctx, ctx->kl.attn_counters) : (int*)nullptr, fused ? out : (float*)nullptr,
                fused ? planes : (__nv_bfloat16*)nullptr, row_base, n_rows_fixed, pos0_fixed));
    return SWIFT_OK;
}

// Attention of one block for the forward chunk's rows: split kernel + merge of the splits into `out` (fp32 rows)
// and, when given, the hi/lo planes the next GEMM reads.  `full_model`: no sub-layer of this forward is skipped.  Where
// a tensor-core kernel is in use for decoding, the target model's forwards (verification of a chain, vanilla steps) all take
// the same one (grouped-query models: the tile kernel, which their layer-skipped forwards take as well; SWIFT_ATTN_MMA=1: the
// swapped kernel, layer-skipped forwards on the streaming one); a row's result never depends on the row count within either family, which is what makes a
// vanilla step and the same row of a verification agree bit for bit.
template <typename T>
swift_status launch_attn(swift_ctx* ctx, int rows, const int* page_table, int block, float* out, __nv_bfloat16* planes,
                         bool full_model)
{
    const swift_model_desc& d = ctx->d;
    if ((full_model || ctx->attn_tile_drafts) && ctx->attn_tile_decode && !ctx->tree_forward) {
        ST(launch_attn_tile<T>(ctx, page_table, block, rows, (int)ROWS, 0, 0, 0));
        CU(launch_k(attn_combine_kernel, dim3(d.n_heads, rows), dim3(d.head_dim), 2 * (size_t)ctx->max_splits * sizeof(float), ctx,
                    (const DevState*)state_of(ctx), (const float*)kptr<float>(ctx, ctx->kl.o_part),
                    (const float2*)kptr<float2>(ctx, ctx->kl.ml_part), ctx->max_splits, d.n_heads, d.head_dim, out, planes, (int)ROWS, 0, 0, 0, 1));
        return SWIFT_OK;
    }
    if (d.head_dim == 128 && full_model && ctx->attn_mma) {
        const bool fused = rows == 1 && ctx->fuse_combine;
        const swift_status ms = (d.n_heads / d.n_kv_heads) * rows <= 8 ? launch_attn_mma<T, 1>(ctx, page_table, block, fused, out, planes)
                                                                       : launch_attn_mma<T, 2>(ctx, page_table, block, fused, out, planes);
        if (ms != SWIFT_OK) return ms;
        if (fused) return SWIFT_OK;
        CU(launch_k(attn_combine_kernel, dim3(d.n_heads, rows), dim3(d.head_dim), 2 * (size_t)ctx->max_splits * sizeof(float), ctx,
                    (const DevState*)state_of(ctx), (const float*)kptr<float>(ctx, ctx->kl.o_part),
                    (const float2*)kptr<float2>(ctx, ctx->kl.ml_part), ctx->max_splits, d.n_heads, d.head_dim, out, planes, (int)ROWS, 0, 0, 0, 1));
        return SWIFT_OK;
    }
    // The streaming kernel (head_dim 128) takes the rows in groups of at most attn_rows_per_cta, one group per
    // grid.z slice: fewer rows per CTA means fewer registers and more CTAs in flight.
    int mr = attn_mr_of(rows), groups = 1;
    if (d.head_dim == 128 && rows > ctx->attn_rows_per_cta) {
        mr = ctx->attn_rows_per_cta;
        groups = ceil_div(rows, mr);
    }
    const bool fused = d.head_dim == 128 && rows == 1 && ctx->fuse_combine;
    float* fo = fused ? out : nullptr;
    __nv_bfloat16* fp = fused ? planes : nullptr;
    swift_status s;
    switch (mr) {
    case 1: s = launch_attn_mr<T, 1>(ctx, page_table, block, groups, fo, fp); break;
    case 2: s = launch_attn_mr<T, 2>(ctx, page_table, block, groups, fo, fp); break;
    case 4: s = launch_attn_mr<T, 4>(ctx, page_table, block, groups, fo, fp); break;
    case 6: s = launch_attn_mr<T, 6>(ctx, page_table, block, groups, fo, fp); break;
    case 8: s = launch_attn_mr<T, 8>(ctx, page_table, block, groups, fo, fp); break;
    case 12: s = launch_attn_mr<T, 12>(ctx, page_table, block, groups, fo, fp); break;
    default: s = launch_attn_mr<T, 16>(ctx, page_table, block, groups, fo, fp); break;
    }
    if (s != SWIFT_OK || fused) return s;
    CU(launch_k(attn_combine_kernel, dim3(d.n_heads, rows), dim3(d.head_dim), 2 * (size_t)ctx->max_splits * sizeof(float), ctx,
                (const DevState*)state_of(ctx), (const float*)kptr<float>(ctx, ctx->kl.o_part),
                (const float2*)kptr<float2>(ctx, ctx->kl.ml_part), ctx->max_splits, d.n_heads, d.head_dim, out, planes, (int)ROWS, 0, 0, 0, 1));
    return SWIFT_OK;
}

struct HeadOpts {
    bool run = false;
    int mode = VOCAB_PLAIN;
};

// Where a draft step leaves its top predictions when dynamic verification is on (greedy decoding only), else null.
int* tree_cand(swift_ctx* ctx, const HeadOpts& head)
{
    return (head.mode == VOCAB_DRAFT && ctx->tree_rows > 0 && ctx->mode == SWIFT_GREEDY) ? kptr<int>(ctx, ctx->kl.cand) : nullptr;
}


// Enqueues the kernels of one forward chunk of at most `rows` (<= 16) rows.  The device state
// (pos0, n_rows, tok_off) must have been set by a preceding kernel on the same stream.
template <typename T, typename TKV>
swift_status forward_chunk(swift_ctx* ctx, int rows, const int* toks_dev, const uint8_t* skip, const int* page_table,
                           HeadOpts head)
{
    const swift_model_desc& d = ctx->d;
    DevState* st = state_of(ctx);
    const int mr = mr_of(rows);
    const int dm = d.d_model, qd = d.n_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, nqkv = qd + 2 * kd;
    float* h = kptr<float>(ctx, ctx->kl.h);
    float* xn = kptr<float>(ctx, ctx->kl.xn);
    float* xa = kptr<float>(ctx, ctx->kl.xa);
    float* act = kptr<float>(ctx, ctx->kl.act);
    float* part = kptr<float>(ctx, ctx->kl.part);
    const bool tc = ctx->use_tc;
    __nv_bfloat16* xn_hl = tc ? kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl) : nullptr;
    __nv_bfloat16* xa_hl = tc ? kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl) : nullptr;
    __nv_bfloat16* act_hl = tc ? kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl) : nullptr;
    const float* pend = nullptr;      // pending residual-branch output (split-K slabs) not yet added to h
    int pend_S = 0, S = 0;
    bool full_model = true;
    for (int sl = 0; sl < 2 * d.n_blocks; ++sl) full_model = full_model && !(skip && skip[sl]);

    CU(launch_k(embed_kernel<T>, dim3(rows), dim3(256), 0, ctx, st, toks_dev, (const T*)wptr<T>(ctx, ctx->wl.embed), h, dm, d.vocab));
    for (int b = 0; b < d.n_blocks; ++b) {
        if (!(skip && skip[2 * b])) {
            CU(launch_k(resid_norm_kernel, dim3(rows), dim3(512), 0, ctx, (const DevState*)st, h, pend, pend_S, (size_t)ROWS * dm,
                        (const float*)wptr<float>(ctx, ctx->wl.attn_norm[b]), xn, xn_hl, dm, d.rms_eps));
            ST(run_gemm<T>(ctx, mr, GemmSite{xn, nqkv, dm, wptr<T>(ctx, ctx->wl.wqkv[b]), tc ? &ctx->tm_wqkv[b] : nullptr, &ctx->tm_xn}, &S));
            CU(launch_k(qkv_post_kernel<TKV>, dim3(rows, d.n_heads + 2 * d.n_kv_heads), dim3(d.head_dim / 2), 0, ctx,
                        (const DevState*)st, (const float*)part, S, (size_t)ROWS * nqkv, nqkv, kptr<float>(ctx, ctx->kl.q),
                        reinterpret_cast<TKV*>(ctx->kvbase), page_table, ctx->kv, b, d.n_heads,
                        (const float2*)kptr<float2>(ctx, ctx->kl.rope), d.max_positions));
            ST(launch_attn<TKV>(ctx, rows, page_table, b, xa, xa_hl, full_model));
            ST(run_gemm<T>(ctx, mr, GemmSite{xa, dm, qd, wptr<T>(ctx, ctx->wl.wo[b]), tc ? &ctx->tm_wo[b] : nullptr, &ctx->tm_xa}, &S));
            pend = part; pend_S = S;
        }
        if (!(skip && skip[2 * b + 1])) {
            CU(launch_k(resid_norm_kernel, dim3(rows), dim3(512), 0, ctx, (const DevState*)st, h, pend, pend_S, (size_t)ROWS * dm,
                        (const float*)wptr<float>(ctx, ctx->wl.mlp_norm[b]), xn, xn_hl, dm, d.rms_eps));
            ST(run_gemm<T>(ctx, mr, GemmSite{xn, 2 * d.ffn, dm, wptr<T>(ctx, ctx->wl.wgu[b]), tc ? &ctx->tm_wgu[b] : nullptr, &ctx->tm_xn}, &S));
            CU(launch_k(swiglu_kernel, dim3(ceil_div(d.ffn, 256), rows), dim3(256), 0, ctx, (const DevState*)st, (const float*)part, S,
                        (size_t)ROWS * 2 * d.ffn, act, act_hl, d.ffn));
            ST(run_gemm<T>(ctx, mr, GemmSite{act, dm, d.ffn, wptr<T>(ctx, ctx->wl.wdown[b]), tc ? &ctx->tm_wdown[b] : nullptr, &ctx->tm_act}, &S));
            pend = part; pend_S = S;
        }
    }
    if (head.run) {
        CU(launch_k(resid_norm_kernel, dim3(rows), dim3(512), 0, ctx, (const DevState*)st, h, pend, pend_S, (size_t)ROWS * dm,
                    (const float*)wptr<float>(ctx, ctx->wl.final_norm), xn, xn_hl, dm, d.rms_eps));
        ST(run_gemm<T>(ctx, mr, GemmSite{xn, d.vocab, dm, wptr<T>(ctx, ctx->wl.lm_head), &ctx->tm_lm_head, &ctx->tm_xn}, &S));
        CU(launch_k(vocab_kernel, dim3(rows), dim3(VOCAB_THREADS), vocab_cache_bytes(ctx), ctx, st, (const float*)part, S, (size_t)ROWS * d.vocab,
                    kptr<float>(ctx, ctx->kl.logits), d.vocab, 1.0f / ctx->temperature, head.mode,
                    sampling_flag(ctx), kptr<float>(ctx, ctx->kl.q_rows), ctx->top_p, vocab_cache_bytes(ctx) != 0 ? 1 : 0,
                    tree_cand(ctx, head), kptr<int>(ctx, ctx->kl.cand_n)));
    }
    CU(cudaGetLastError());
    return SWIFT_OK;
}

// The same walk on the tensor-core path, with the element-wise steps folded into the GEMM epilogues:
// per block  QKV GEMM (+RMSNorm scale, RoPE, KV append) -> attention split -> combine -> o_proj GEMM
// (+residual, next norm's planes) -> gate/up GEMM (+RMSNorm scale, SwiGLU) -> down GEMM (+residual ...).
template <typename TKV>
swift_status forward_chunk_fused(swift_ctx* ctx, int rows, const int* toks_dev, const uint8_t* skip, const int* page_table,
                                 HeadOpts head)
{
    typedef __nv_bfloat16 T;
    const swift_model_desc& d = ctx->d;
    DevState* st = state_of(ctx);
    const int mr = mr_of(rows);
    const int dm = d.d_model, qd = d.n_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, nqkv = qd + 2 * kd;
    float* h = kptr<float>(ctx, ctx->kl.h);
    float* xa = kptr<float>(ctx, ctx->kl.xa);
    __nv_bfloat16* xn_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
    __nv_bfloat16* xa_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl);
    __nv_bfloat16* act_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl);
    float* sumsq = kptr<float>(ctx, ctx->kl.sumsq);

    std::vector<int> kept;                       // sub-layers that run, in walk order
    for (int sl = 0; sl < 2 * d.n_blocks; ++sl)
        if (!(skip && skip[sl])) kept.push_back(sl);
    const bool full_model = (int)kept.size() == 2 * d.n_blocks;
    auto gain_of = [&](size_t k) -> const float* {   // gain of the RMSNorm in front of kept[k]; past the end: the final norm
        if (k < kept.size()) return wptr<float>(ctx, (kept[k] & 1) ? ctx->wl.mlp_norm[kept[k] >> 1] : ctx->wl.attn_norm[kept[k] >> 1]);
        return head.run ? wptr<float>(ctx, ctx->wl.final_norm) : nullptr;
    };
    EpiParams base;
    memset(&base, 0, sizeof base);
    base.inv_d = 1.0f / (float)dm;
    base.eps = d.rms_eps;
    base.sumsq_in = sumsq;
    base.sum_rows = ROWS;
    int n_tiles_in = 1;                          // the embedding gather writes one "tile" of sums

    // the weight matrices in the order this forward streams them: each GEMM prefetches the start of the next one
    struct NextW { const CUtensorMap* map; int N, K; };
    std::vector<NextW> order;
    for (int sl : kept) {
        const int b = sl >> 1;
        if (!(sl & 1)) {
            order.push_back({&ctx->tm_wqkv[b], nqkv, dm});
            order.push_back({&ctx->tm_wo[b], dm, qd});
        } else {
            order.push_back({&ctx->tm_wgu[b], 2 * d.ffn, dm});
            order.push_back({&ctx->tm_wdown[b], dm, d.ffn});
        }
    }
    if (head.run) order.push_back({&ctx->tm_lm_head, d.vocab, dm});
    size_t gemm_index = 0;
    auto gemm = [&](int epi, const CUtensorMap* mw, const CUtensorMap* mx, int N, int K, const EpiParams& ep_in) -> swift_status {
        EpiParams ep = ep_in;
        const CUtensorMap* next_map = nullptr;
        ++gemm_index;
        if (ctx->prefetch_next && gemm_index < order.size()) {
            next_map = order[gemm_index].map;
            ep.next_N = order[gemm_index].N;
            ep.next_K = order[gemm_index].K;
            ep.next_tiles = ctx->prefetch_tiles;
        }
        const GemmSite g{nullptr, N, K, nullptr, mw, mx};
        switch (epi) {
        case EPI_QKV: return launch_gemm_tc<EPI_QKV, TKV>(ctx, g, ep, next_map);
        case EPI_SWIGLU: return launch_gemm_tc<EPI_SWIGLU, float>(ctx, g, ep, next_map);
        case EPI_RESID: return launch_gemm_tc<EPI_RESID, float>(ctx, g, ep, next_map);
        default: return launch_gemm_tc<EPI_PLAIN, float>(ctx, g, ep, next_map);
        }
    };

    CU(launch_k(embed_fused_kernel<T>, dim3(rows), dim3(1024), 0, ctx, st, toks_dev, (const T*)wptr<T>(ctx, ctx->wl.embed), h,
                gain_of(0), xn_hl, sumsq, dm, d.vocab));
    const int d_tiles = ceil_div(dm, TC_TILE_N);
    for (size_t k = 0; k < kept.size(); ++k) {
        const int b = kept[k] >> 1;
        EpiParams resid = base;
        resid.h = h; resid.gain_next = gain_of(k + 1); resid.planes_out = xn_hl; resid.sumsq_out = sumsq;
        if (!(kept[k] & 1)) {
            EpiParams ep = base;
            ep.n_sumsq_tiles = n_tiles_in;
            ep.q_out = kptr<float>(ctx, ctx->kl.q); ep.kv_pool = ctx->kvbase; ep.page_table = page_table; ep.L = ctx->kv;
            ep.block = b; ep.n_heads = d.n_heads; ep.max_positions = d.max_positions; ep.rope_cs = kptr<float2>(ctx, ctx->kl.rope);
            ST(gemm(EPI_QKV, &ctx->tm_wqkv[b], &ctx->tm_xn, nqkv, dm, ep));
            ST(launch_attn<TKV>(ctx, rows, page_table, b, xa, xa_hl, full_model));
            ST(gemm(EPI_RESID, &ctx->tm_wo[b], &ctx->tm_xa, dm, qd, resid));
        } else {
            EpiParams ep = base;
            ep.n_sumsq_tiles = n_tiles_in;
            ep.act_planes = act_hl; ep.ffn = d.ffn;
            ST(gemm(EPI_SWIGLU, &ctx->tm_wgu[b], &ctx->tm_xn, 2 * d.ffn, dm, ep));
            ST(gemm(EPI_RESID, &ctx->tm_wdown[b], &ctx->tm_act, dm, d.ffn, resid));
        }
        n_tiles_in = d_tiles;
    }
    if (head.run) {
        EpiParams ep = base;
        ep.n_sumsq_tiles = n_tiles_in;
        ST(gemm(EPI_PLAIN, &ctx->tm_lm_head, &ctx->tm_xn, d.vocab, dm, ep));
        CU(launch_k(vocab_kernel, dim3(rows), dim3(VOCAB_THREADS), vocab_cache_bytes(ctx), ctx, st, (const float*)kptr<float>(ctx, ctx->kl.part), 1,
                    (size_t)ROWS * d.vocab, kptr<float>(ctx, ctx->kl.logits), d.vocab, 1.0f / ctx->temperature, head.mode,
                    sampling_flag(ctx), kptr<float>(ctx, ctx->kl.q_rows), ctx->top_p, vocab_cache_bytes(ctx) != 0 ? 1 : 0,
                    tree_cand(ctx, head), kptr<int>(ctx, ctx->kl.cand_n)));
    }
    CU(cudaGetLastError());
    return SWIFT_OK;
}

// The full model over a chunk of up to TC_BIG_ROWS rows (prefill): the same walk as forward_chunk_fused with every weight
// tile applied to all rows at once (the GEMM in its NB = 8 form, tensor-core attention over all rows of a chunk per K,V
// load), no output head.  Tokens in the big_tok device array; the control block holds pos0 and the row count.
template <typename TKV>
swift_status forward_chunk_big(swift_ctx* ctx, int rows, const int* page_table)
{
    typedef __nv_bfloat16 T;
    constexpr int NB = TC_NB_MAX;
    const swift_model_desc& d = ctx->d;
    DevState* st = state_of(ctx);
    const int dm = d.d_model, qd = d.n_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, nqkv = qd + 2 * kd;
    float* h = kptr<float>(ctx, ctx->kl.h);
    float* xa = kptr<float>(ctx, ctx->kl.xa);
    __nv_bfloat16* xn_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
    __nv_bfloat16* xa_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl);
    __nv_bfloat16* act_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl);
    float* sumsq = kptr<float>(ctx, ctx->kl.sumsq);
    EpiParams base;
    memset(&base, 0, sizeof base);
    base.inv_d = 1.0f / (float)dm;
    base.eps = d.rms_eps;
    base.sumsq_in = sumsq;
    base.sum_rows = TC_BIG_ROWS;
    const int n_prob = ceil_div(rows, TC_ROWS_MAX);      // row ranges of 128 that each GEMM launch runs as separate problems
    const int d_tiles = ceil_div(dm, TC_TILE_N);
    int n_tiles_in = 1;
    CU(launch_k(embed_fused_kernel<T>, dim3(rows), dim3(1024), 0, ctx, st, (const int*)kptr<int>(ctx, ctx->kl.big_tok),
                (const T*)wptr<T>(ctx, ctx->wl.embed), h, (const float*)wptr<float>(ctx, ctx->wl.attn_norm[0]), xn_hl, sumsq, dm, d.vocab));
    for (int b = 0; b < d.n_blocks; ++b) {
        EpiParams ep = base;
        ep.n_sumsq_tiles = n_tiles_in;
        ep.q_out = kptr<float>(ctx, ctx->kl.q); ep.kv_pool = ctx->kvbase; ep.page_table = page_table; ep.L = ctx->kv;
        ep.block = b; ep.n_heads = d.n_heads; ep.max_positions = d.max_positions; ep.rope_cs = kptr<float2>(ctx, ctx->kl.rope);
        ST((launch_gemm_tc<EPI_QKV, TKV, NB>(ctx, GemmSite{nullptr, nqkv, dm, nullptr, &ctx->tm_wqkv[b], &ctx->tm_xn_big}, ep, nullptr, n_prob)));
        if (ctx->attn_tile) ST((launch_attn_tile<TKV>(ctx, page_table, b, rows, TC_BIG_ROWS, 0, 0, 0)));
        else ST((launch_attn_mma<TKV, 2>(ctx, page_table, b, false, xa, xa_hl, TC_BIG_ROWS, 0, 0, 0,
                                         ceil_div((d.n_heads / d.n_kv_heads) * rows, 16))));
        CU(launch_k(attn_combine_kernel, dim3(d.n_heads, rows), dim3(d.head_dim), 2 * (size_t)ctx->max_splits * sizeof(float), ctx,
                    (const DevState*)st, (const float*)kptr<float>(ctx, ctx->kl.o_part), (const float2*)kptr<float2>(ctx, ctx->kl.ml_part),
                    ctx->max_splits, d.n_heads, d.head_dim, xa, xa_hl, (int)TC_BIG_ROWS, 0, 0, 0, 1));
        EpiParams resid = base;
        resid.h = h; resid.planes_out = xn_hl; resid.sumsq_out = sumsq;
        resid.gain_next = wptr<float>(ctx, ctx->wl.mlp_norm[b]);
        ST((launch_gemm_tc<EPI_RESID, float, NB>(ctx, GemmSite{nullptr, dm, qd, nullptr, &ctx->tm_wo[b], &ctx->tm_xa_big}, resid, nullptr, n_prob)));
        EpiParams sw = base;
        sw.n_sumsq_tiles = d_tiles;
        sw.act_planes = act_hl; sw.ffn = d.ffn;
        ST((launch_gemm_tc<EPI_SWIGLU, float, NB>(ctx, GemmSite{nullptr, 2 * d.ffn, dm, nullptr, &ctx->tm_wgu[b], &ctx->tm_xn_big}, sw, nullptr, n_prob)));
        // nothing reads the residual stream of a prefill chunk after its last block: no planes, no sums there
        resid.gain_next = b + 1 < d.n_blocks ? wptr<float>(ctx, ctx->wl.attn_norm[b + 1]) : nullptr;
        ST((launch_gemm_tc<EPI_RESID, float, NB>(ctx, GemmSite{nullptr, dm, d.ffn, nullptr, &ctx->tm_wdown[b], &ctx->tm_act_big}, resid, nullptr, n_prob)));
        n_tiles_in = d_tiles;
    }
    CU(cudaGetLastError());
    return SWIFT_OK;
}

swift_status forward_chunk_any(swift_ctx* ctx, int rows, const int* toks_dev, const uint8_t* skip, const int* page_table,
                               HeadOpts head)
{
    if (ctx->use_tc && ctx->fuse) {
        if (ctx->d.kv_dtype == SWIFT_BF16) return forward_chunk_fused<__nv_bfloat16>(ctx, rows, toks_dev, skip, page_table, head);
        return forward_chunk_fused<float>(ctx, rows, toks_dev, skip, page_table, head);
    }
    if (ctx->d.dtype == SWIFT_BF16) {
        if (ctx->d.kv_dtype == SWIFT_BF16) return forward_chunk<__nv_bfloat16, __nv_bfloat16>(ctx, rows, toks_dev, skip, page_table, head);
        return forward_chunk<__nv_bfloat16, float>(ctx, rows, toks_dev, skip, page_table, head);
    }
    return forward_chunk<float, float>(ctx, rows, toks_dev, skip, page_table, head);
}

// A forward chunk depends on the host only through (rows, skip mask, page table, token source, head
// options, sampling settings); everything else it reads from the device control block.  So its launch
// sequence is captured once into a CUDA graph and replayed: one graph launch instead of several
// hundred kernel launches per forward.
struct FwdKey {
    int rows, head_run, head_mode, sampling, use_tc, use_pdl, fuse, tree;
    float temperature, top_p;
    const void* toks;
    const void* page_table;
    std::vector<uint8_t> mask;
    bool operator==(const FwdKey& o) const
    {
        return rows == o.rows && head_run == o.head_run && head_mode == o.head_mode && sampling == o.sampling &&
               use_tc == o.use_tc && use_pdl == o.use_pdl && fuse == o.fuse && tree == o.tree && temperature == o.temperature && top_p == o.top_p && toks == o.toks && page_table == o.page_table && mask == o.mask;
    }
};
struct FwdGraph {
    FwdKey key;
    cudaGraphExec_t exec;
    int64_t launches;
    uint64_t last_use;
};

swift_status forward_cached(swift_ctx* ctx, int rows, const int* toks_dev, const uint8_t* skip, const int* page_table,
                            HeadOpts head)
{
    if (!ctx->use_graphs) return forward_chunk_any(ctx, rows, toks_dev, skip, page_table, head);
    const int L = 2 * ctx->d.n_blocks;
    FwdKey key{rows, head.run ? 1 : 0, head.mode, sampling_flag(ctx), ctx->use_tc ? 1 : 0, ctx->use_pdl ? 1 : 0, ctx->fuse ? 1 : 0, (tree_cand(ctx, head) ? 1 : 0) | (ctx->tree_forward ? 2 : 0), ctx->temperature, ctx->top_p, toks_dev, page_table,
               skip ? std::vector<uint8_t>(skip, skip + L) : std::vector<uint8_t>()};
    auto& cache = *ctx->graphs;
    ctx->graph_clock++;
    for (auto& g : cache)
        if (g.key == key) {
            g.last_use = ctx->graph_clock;
            CU(cudaGraphLaunch(g.exec, ctx->stream));
            ctx->launches += g.launches;
            return SWIFT_OK;
        }
    // capture a new one
    const int64_t before = ctx->launches;
    cudaGraph_t graph = nullptr;
    CU(cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
    const swift_status fs = forward_chunk_any(ctx, rows, toks_dev, skip, page_table, head);
    const cudaError_t ce = cudaStreamEndCapture(ctx->stream, &graph);
    if (fs != SWIFT_OK) { if (graph) cudaGraphDestroy(graph); return fs; }
    if (ce != cudaSuccess) return fail(ctx, SWIFT_ECUDA, "stream capture failed: %s", cudaGetErrorString(ce));
    if (getenv("SWIFT_DEBUG_GRAPH")) {       // how many of the captured dependencies are programmatic (PDL) edges
        size_t n_nodes = 0, n_edges = 0;
        cudaGraphGetNodes(graph, nullptr, &n_nodes);
        cudaGraphGetEdges_v2(graph, nullptr, nullptr, nullptr, &n_edges);
        std::vector<cudaGraphNode_t> from(n_edges), to(n_edges);
        std::vector<cudaGraphEdgeData> data(n_edges);
        size_t n_prog = 0;
        if (n_edges && cudaGraphGetEdges_v2(graph, from.data(), to.data(), data.data(), &n_edges) == cudaSuccess)
            for (size_t i = 0; i < n_edges; ++i) n_prog += data[i].type == cudaGraphDependencyTypeProgrammatic ? 1 : 0;
        fprintf(stderr, "[swift] captured forward: %zu nodes, %zu edges, %zu programmatic\n", n_nodes, n_edges, n_prog);
    }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess) return fail(ctx, SWIFT_ECUDA, "graph instantiation failed: %s", cudaGetErrorString(ie));
    const int64_t n_launch = ctx->launches - before;
    ctx->launches = before;
    if (cache.size() >= 24) {             // evict the least recently used graph
        size_t victim = 0;
        for (size_t i = 1; i < cache.size(); ++i) if (cache[i].last_use < cache[victim].last_use) victim = i;
        cudaGraphExecDestroy(cache[victim].exec);
        cache.erase(cache.begin() + victim);
    }
    cache.push_back(FwdGraph{key, exec, n_launch, ctx->graph_clock});
    CU(cudaGraphLaunch(exec, ctx->stream));
    ctx->launches += n_launch;
    return SWIFT_OK;
}

} // namespace

// =============================================================================== helpers
namespace {

struct HostState { DevState s; };

swift_status read_state(swift_ctx* ctx, DevState* out)
{
    CU(copy_async(ctx, out, state_of(ctx), sizeof(DevState), cudaMemcpyDeviceToHost));
    CU(cudaStreamSynchronize(ctx->stream));
    ctx->last_state = *out;
    if (out->error) {
        const int code = out->error;
        CU(cudaMemsetAsync(&state_of(ctx)->error, 0, sizeof(int), ctx->stream));
        if (code == TC_ERR_TIMEOUT) {
            CU(cudaMemsetAsync(kptr<int>(ctx, ctx->kl.counters), 0, TC_MAX_TILES * 4, ctx->stream));
            return fail(ctx, SWIFT_ETIMEOUT, "a bounded wait inside the tensor-core GEMM ran out");
        }
        if (code == 3) return fail(ctx, SWIFT_ETIMEOUT, "a bounded wait inside the attention kernel ran out");
        return fail(ctx, SWIFT_EINVAL, "device reported an invalid token id");
    }
    return SWIFT_OK;
}

const int* pt_main(swift_ctx* c) { return kptr<int>(c, c->kl.pt_main); }
const int* pt_score(swift_ctx* c) { return kptr<int>(c, c->kl.pt_score); }

// Redirects the pages that hold positions [p_begin, p_end) to scratch pages in the scoring page
// table, copying the first page when the range starts inside it (copy-on-write).
swift_status prepare_scratch(swift_ctx* ctx, int p_begin, int p_end)
{
    const int P = ctx->d.page_size;
    const int first = p_begin / P, last = (p_end - 1) / P;
    if (last - first + 1 > ctx->n_pages_scratch) return fail(ctx, SWIFT_ECAPACITY, "window spans too many KV pages");
    std::vector<int> pt(ctx->n_pages_main);
    for (int i = 0; i < ctx->n_pages_main; ++i) pt[i] = i;
    for (int p = first; p <= last; ++p) pt[p] = ctx->n_pages_main + (p - first);
    CU(copy_async(ctx, kptr<int>(ctx, ctx->kl.pt_score), pt.data(), pt.size() * 4, cudaMemcpyHostToDevice));
    if (p_begin % P) {
        const size_t v16 = page_bytes(&ctx->d) / 16;
        page_copy_kernel<<<296, 256, 0, ctx->stream>>>(reinterpret_cast<uint4*>(ctx->kvbase), v16, first, ctx->n_pages_main);
        ctx->launches++;
        CU(cudaGetLastError());
    }
    return SWIFT_OK;
}

// head_mode: 0 = no output head, 1 = last chunk only, 2 = every chunk.
swift_status run_rows(swift_ctx* ctx, const int32_t* tokens, int n_rows, int pos0, const uint8_t* skip,
                      const int* page_table, int head_mode, float* logits_host, int32_t* argmax_host, int* last_chunk_rows)
{
    DevState* st = state_of(ctx);
    for (int c0 = 0; c0 < n_rows; c0 += ROWS) {
        const int rows = std::min(ROWS, n_rows - c0);
        const bool last = c0 + rows == n_rows;
        CU(copy_async(ctx, st->row_tok, tokens + c0, rows * 4, cudaMemcpyHostToDevice));
        set_rows_kernel<<<1, 1, 0, ctx->stream>>>(st, pos0 + c0, rows);
        ctx->launches++;
        HeadOpts head;
        head.run = head_mode == 2 || (head_mode == 1 && last);
        ST(forward_cached(ctx, rows, st->row_tok, skip, page_table, head));
        if (head.run && logits_host)
            CU(copy_async(ctx, logits_host + (size_t)c0 * ctx->d.vocab, kptr<float>(ctx, ctx->kl.logits),
                               (size_t)rows * ctx->d.vocab * 4, cudaMemcpyDeviceToHost));
        if (head.run && argmax_host)
            CU(copy_async(ctx, argmax_host + c0, st->argmax, rows * 4, cudaMemcpyDeviceToHost));
        if (last && last_chunk_rows) *last_chunk_rows = rows;
    }
    return SWIFT_OK;
}

swift_status check_tokens(swift_ctx* ctx, const int32_t* t, int n)
{
    if (!t) return fail(ctx, SWIFT_EINVAL, "null token pointer");
    for (int i = 0; i < n; ++i)
        if (t[i] < 0 || t[i] >= ctx->d.vocab) return fail(ctx, SWIFT_EINVAL, "token id %d at index %d outside [0, %d)", t[i], i, ctx->d.vocab);
    return SWIFT_OK;
}

void launch_begin_round(swift_ctx* ctx, float stop_conf)
{
    begin_round_kernel<<<1, 1, 0, ctx->stream>>>(state_of(ctx), ctx->pending, 1, ctx->round, stop_conf, (unsigned)ctx->seed,
                                                 (unsigned)(ctx->seed >> 32));
    ctx->launches++;
}

// ---- enqueue-only forms of the steps (no host synchronisation); used by the entry points and by generate
swift_status enqueue_draft(swift_ctx* ctx, const uint8_t* skip, int max_k, float stop_conf)
{
    DevState* st = state_of(ctx);
    ctx->round++;
    launch_begin_round(ctx, stop_conf);
    for (int j = 1; j <= max_k; ++j) {
        begin_draft_step_kernel<<<1, 1, 0, ctx->stream>>>(st, ctx->n, j);
        ctx->launches++;
        HeadOpts head;
        head.run = true; head.mode = VOCAB_DRAFT;
        ST(forward_cached(ctx, 1, st->draft_tok, skip, pt_main(ctx), head));
    }
    ctx->last_max_k = max_k;
    ctx->round_open = true;
    return SWIFT_OK;
}

// Dynamic verification applies to rounds of greedy decoding that verify what the device drafted.
bool tree_active(const swift_ctx* ctx) { return ctx->tree_rows > 0 && ctx->mode == SWIFT_GREEDY; }

swift_status enqueue_verify(swift_ctx* ctx, int rows_launch, int forced_k)
{
    DevState* st = state_of(ctx);
    if (forced_k < 0 && tree_active(ctx)) {
        // the chain plus the draft model's next-best predictions, as many rows as the budget holds
        const int budget = std::max(ctx->tree_rows, rows_launch);
        begin_verify_tree_kernel<<<1, 1, 0, ctx->stream>>>(st, ctx->n, kptr<int>(ctx, ctx->kl.cand), kptr<int>(ctx, ctx->kl.cand_n), budget);
        rows_launch = budget;
        ctx->tree_forward = true;
    } else {
        begin_verify_kernel<<<1, 1, 0, ctx->stream>>>(st, ctx->n, forced_k);
    }
    ctx->launches++;
    HeadOpts head;
    head.run = true;
    const swift_status fs = forward_cached(ctx, rows_launch, st->draft_tok, nullptr, pt_main(ctx), head);
    ctx->tree_forward = false;
    return fs;
}

swift_status enqueue_accept(swift_ctx* ctx)
{
    accept_kernel<<<1, VOCAB_THREADS, 0, ctx->stream>>>(state_of(ctx), kptr<float>(ctx, ctx->kl.logits),
                                                        kptr<float>(ctx, ctx->kl.q_rows), ctx->d.vocab,
                                                        ctx->mode == SWIFT_SAMPLING ? 1 : 0, 1.0f / ctx->temperature,
                                                        ctx->seed, (uint32_t)ctx->round);
    ctx->launches++;
    if (ctx->tree_rows > 0) {             // an accepted alternative is moved to the cache slot of its depth (no-op for a chain)
        if (ctx->d.kv_dtype == SWIFT_BF16)
            kv_move_accepted_kernel<__nv_bfloat16><<<dim3(ctx->d.n_blocks, 2), 256, 0, ctx->stream>>>(
                state_of(ctx), reinterpret_cast<__nv_bfloat16*>(ctx->kvbase), pt_main(ctx), ctx->kv, ctx->n);
        else
            kv_move_accepted_kernel<float><<<dim3(ctx->d.n_blocks, 2), 256, 0, ctx->stream>>>(
                state_of(ctx), reinterpret_cast<float*>(ctx->kvbase), pt_main(ctx), ctx->kv, ctx->n);
        ctx->launches++;
    }
    CU(cudaGetLastError());
    return SWIFT_OK;
}

// Folds the outcome of a round (read back from the device) into the host-side committed state.
void commit_round(swift_ctx* ctx, const DevState& hs)
{
    const int a = hs.n_accepted;
    for (int j = 1; j <= a; ++j) ctx->hist.push_back(hs.draft_tok[j]);
    ctx->hist.push_back(hs.next_token);
    ctx->n += a + 1;
    ctx->pending = hs.next_token;
    ctx->phase = PH_READY;
    ctx->round_open = false;
}

// Scores C candidates; results (match counts) land in the score_out device array.
template <typename TKV>
swift_status enqueue_score_batched(swift_ctx* ctx, const uint8_t* masks, int C, int gamma);

swift_status enqueue_score(swift_ctx* ctx, const uint8_t* masks, int C, int gamma)
{
    if (ctx->batched_scoring) {                        // all candidates side by side where the shape allows it
        const swift_status bs = ctx->d.kv_dtype == SWIFT_BF16 ? enqueue_score_batched<__nv_bfloat16>(ctx, masks, C, gamma)
                                                              : enqueue_score_batched<float>(ctx, masks, C, gamma);
        if (bs != SWIFT_EUNSUPPORTED) return bs;
    }
    const int n = ctx->n, L = 2 * ctx->d.n_blocks;
    DevState* st = state_of(ctx);
    int* tok_dev = kptr<int>(ctx, ctx->kl.score_tok);
    int* truth_dev = kptr<int>(ctx, ctx->kl.score_truth);
    int* out_dev = kptr<int>(ctx, ctx->kl.score_out);
    CU(copy_async(ctx, tok_dev, ctx->hist.data() + (n - gamma), gamma * 4, cudaMemcpyHostToDevice));
    CU(copy_async(ctx, truth_dev, ctx->hist.data() + (n - gamma + 1), gamma * 4, cudaMemcpyHostToDevice));
    ST(prepare_scratch(ctx, n - gamma, n));
    for (int c = 0; c < C; ++c) {
        for (int c0 = 0; c0 < gamma; c0 += ROWS) {
            const int rows = std::min(ROWS, gamma - c0);
            set_rows_kernel<<<1, 1, 0, ctx->stream>>>(st, n - gamma + c0, rows);
            ctx->launches++;
            HeadOpts head;
            head.run = true;
            ST(forward_chunk_any(ctx, rows, tok_dev + c0, masks + (size_t)c * L, pt_score(ctx), head));
            match_count_kernel<<<1, 32, 0, ctx->stream>>>(st, truth_dev + c0, c0 == 0 ? 1 : 0,
                                                          c0 + rows == gamma ? out_dev + c : nullptr);
            ctx->launches++;
        }
    }
    CU(cudaGetLastError());
    return SWIFT_OK;
}

// Bytes one forward must move (weights of the kept sub-layers, output head, cached K,V of the kept attention
// sub-layers, embedding rows in, logits out).  kv_elem_bytes: size of a cached K or V element to count; 0 = as stored.
// The records of a run count 2 bytes (a 16-bit cache, what the method needs); an fp32 cache moves twice that.
// All candidates side by side ("Parallel Candidate Evaluation", Section 4.1): every candidate keeps its own copy of the
// window's gamma residual rows; the sub-layers are walked once, and each is applied to the candidates that keep it,
// gathered into chunks of up to TC_BIG_ROWS rows, so its weights are streamed once per chunk of candidates instead of
// once per 16 rows of every candidate.  Each candidate of a chunk has its own scratch KV pages for the window.  Results
// (match counts) land in the score_out device array.  Returns SWIFT_EUNSUPPORTED when the shape does not fit this form.
template <typename TKV>
swift_status enqueue_score_batched(swift_ctx* ctx, const uint8_t* masks, int C, int gamma)
{
    typedef __nv_bfloat16 T;
    constexpr int NB = TC_NB_MAX;
    const swift_model_desc& d = ctx->d;
    const int n = ctx->n, L = 2 * d.n_blocks, P = d.page_size, pos_w = n - gamma;
    if (!ctx->big_chunks || gamma % ROWS || gamma > TC_ROWS_MAX || C * gamma > SCORE_ROWS_MAX) return SWIFT_EUNSUPPORTED;
    const int pages_per_slot = ceil_div(gamma, P) + 1;
    const int chunk_rows = ctx->many_problems * TC_ROWS_MAX;      // several 128-row problems per GEMM launch
    const int cpg = std::min(std::min(chunk_rows / gamma, ctx->n_pages_scratch / pages_per_slot), (int)SCORE_SLOTS_MAX);   // candidates per chunk
    if (cpg < 1) return SWIFT_EUNSUPPORTED;
    // ---- row maps of the whole round: per sub-layer, the candidates that keep it in chunks of cpg; then the output head
    struct Chunk { int sub; int n_cand; size_t map_off; };
    std::vector<Chunk> chunks;
    std::vector<int> maps;
    for (int sub = 0; sub <= L; ++sub) {
        std::vector<int> keep;
        for (int c = 0; c < C; ++c) if (sub == L || !masks[(size_t)c * L + sub]) keep.push_back(c);
        for (size_t g0 = 0; g0 < keep.size(); g0 += cpg) {
            const int nc = (int)std::min<size_t>(cpg, keep.size() - g0);
            chunks.push_back({sub, nc, maps.size()});
            for (int j = 0; j < nc; ++j)
                for (int i = 0; i < gamma; ++i) maps.push_back(keep[g0 + j] * gamma + i);
            maps.resize(chunks.back().map_off + chunk_rows, 0);
        }
    }
    if (maps.size() > score_map_ints(&d)) return SWIFT_EUNSUPPORTED;
    DevState* st = state_of(ctx);
    int* tok_dev = kptr<int>(ctx, ctx->kl.score_tok);
    int* truth_dev = kptr<int>(ctx, ctx->kl.score_truth);
    int* maps_dev = kptr<int>(ctx, ctx->kl.score_maps);
    float* H_all = kptr<float>(ctx, ctx->kl.score_H);
    CU(copy_async(ctx, tok_dev, ctx->hist.data() + (n - gamma), (size_t)gamma * 4, cudaMemcpyHostToDevice));
    CU(copy_async(ctx, truth_dev, ctx->hist.data() + (n - gamma + 1), (size_t)gamma * 4, cudaMemcpyHostToDevice));
    CU(copy_async(ctx, maps_dev, maps.data(), maps.size() * 4, cudaMemcpyHostToDevice));
    // ---- one page table per candidate slot of a chunk: the window's pages go to the slot's scratch pages
    const int first = pos_w / P, last = (n - 1) / P, np = ctx->n_pages_main;
    std::vector<int> pts((size_t)cpg * np);
    for (int j = 0; j < cpg; ++j) {
        for (int i = 0; i < np; ++i) pts[(size_t)j * np + i] = i;
        for (int p = first; p <= last; ++p) pts[(size_t)j * np + p] = np + j * pages_per_slot + (p - first);
    }
    int* pt_dev = kptr<int>(ctx, ctx->kl.pt_slots);
    CU(copy_async(ctx, pt_dev, pts.data(), pts.size() * 4, cudaMemcpyHostToDevice));
    if (pos_w % P) {                                  // the window starts inside a page: every slot starts from a copy of it
        const size_t v16 = page_bytes(&d) / 16;
        for (int j = 0; j < cpg; ++j) {
            page_copy_kernel<<<296, 256, 0, ctx->stream>>>(reinterpret_cast<uint4*>(ctx->kvbase), v16, first, np + j * pages_per_slot);
            ctx->launches++;
        }
    }
    // ---- the walk
    const int dm = d.d_model, qd = d.n_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, nqkv = qd + 2 * kd;
    float* xa = kptr<float>(ctx, ctx->kl.xa);
    __nv_bfloat16* xn_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
    __nv_bfloat16* xa_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl);
    __nv_bfloat16* act_hl = kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl);
    float* sumsq = kptr<float>(ctx, ctx->kl.sumsq);
    float* logits = kptr<float>(ctx, ctx->kl.score_logits);
    int* pred = kptr<int>(ctx, ctx->kl.score_pred);
    EpiParams base;
    memset(&base, 0, sizeof base);
    base.inv_d = 1.0f / (float)dm;
    base.eps = d.rms_eps;
    base.sumsq_in = sumsq;
    base.sum_rows = TC_BIG_ROWS;
    base.n_sumsq_tiles = 1;                           // gather_norm_kernel leaves each row's sum of squares as tile 0
    embed_rows_kernel<T><<<C * gamma, 256, 0, ctx->stream>>>(st, tok_dev, (const T*)wptr<T>(ctx, ctx->wl.embed), H_all, dm, d.vocab, gamma);
    ctx->launches++;
    for (const Chunk& ch : chunks) {
        const int rows = ch.n_cand * gamma, n_prob = ceil_div(rows, TC_ROWS_MAX);
        const int* map = maps_dev + ch.map_off;
        set_rows_kernel<<<1, 1, 0, ctx->stream>>>(st, pos_w, rows);
        ctx->launches++;
        if (ch.sub == L) {                            // output head: final norm, logits, arg max per row
            gather_norm_kernel<<<rows, 1024, 0, ctx->stream>>>(map, H_all, wptr<float>(ctx, ctx->wl.final_norm), xn_hl, sumsq, dm);
            ctx->launches++;
            ST((launch_gemm_tc_y<NB>(ctx, GemmSite{nullptr, d.vocab, dm, nullptr, &ctx->tm_lm_head, &ctx->tm_xn_big}, base, logits, n_prob)));
            // the head's chunks hold consecutive candidates: their predictions go where their rows are in H_all
            argmax_rows_kernel<<<rows, 1024, 0, ctx->stream>>>(logits, d.vocab, pred + maps[ch.map_off]);
            ctx->launches++;
            continue;
        }
        const int b = ch.sub >> 1;
        EpiParams resid = base;
        resid.h = H_all;                              // the rows' residual stream, in place through the map; nothing chained:
        resid.h_rows = map;                           // the next sub-layer regroups the rows
        if (!(ch.sub & 1)) {
            gather_norm_kernel<<<rows, 1024, 0, ctx->stream>>>(map, H_all, wptr<float>(ctx, ctx->wl.attn_norm[b]), xn_hl, sumsq, dm);
            ctx->launches++;
            EpiParams ep = base;
            ep.q_out = kptr<float>(ctx, ctx->kl.q); ep.kv_pool = ctx->kvbase; ep.page_table = pt_dev; ep.L = ctx->kv;
            ep.block = b; ep.n_heads = d.n_heads; ep.max_positions = d.max_positions; ep.rope_cs = kptr<float2>(ctx, ctx->kl.rope);
            ep.per_block = 1;
            for (int rb = 0; rb < NB * n_prob; ++rb) {
                const int j = std::min((rb * ROWS) / gamma, ch.n_cand - 1);
                ep.rb_pos0[rb] = pos_w + (rb * ROWS) % gamma;
                ep.rb_page_table[rb] = pt_dev + (size_t)j * np;
            }
            ST((launch_gemm_tc<EPI_QKV, TKV, NB>(ctx, GemmSite{nullptr, nqkv, dm, nullptr, &ctx->tm_wqkv[b], &ctx->tm_xn_big}, ep, nullptr, n_prob)));
            // each candidate of the chunk is a sequence of its own behind the context they share
            if (ctx->attn_tile) {
                ST((launch_attn_tile<TKV>(ctx, pt_dev, b, gamma, TC_BIG_ROWS, 0, gamma, pos_w, ch.n_cand, np)));
            } else {
                for (int j = 0; j < ch.n_cand; ++j)
                    ST((launch_attn_mma<TKV, 2>(ctx, pt_dev + (size_t)j * np, b, false, xa, xa_hl, TC_BIG_ROWS, j * gamma, gamma, pos_w,
                                                ceil_div((d.n_heads / d.n_kv_heads) * gamma, 16))));
            }
            CU(launch_k(attn_combine_kernel, dim3(d.n_heads, ch.n_cand * gamma), dim3(d.head_dim), 2 * (size_t)ctx->max_splits * sizeof(float), ctx,
                        (const DevState*)st, (const float*)kptr<float>(ctx, ctx->kl.o_part), (const float2*)kptr<float2>(ctx, ctx->kl.ml_part),
                        ctx->max_splits, d.n_heads, d.head_dim, xa, xa_hl, (int)TC_BIG_ROWS, 0, gamma, pos_w, ch.n_cand));
            ST((launch_gemm_tc<EPI_RESID, float, NB>(ctx, GemmSite{nullptr, dm, qd, nullptr, &ctx->tm_wo[b], &ctx->tm_xa_big}, resid, nullptr, n_prob)));
        } else {
            gather_norm_kernel<<<rows, 1024, 0, ctx->stream>>>(map, H_all, wptr<float>(ctx, ctx->wl.mlp_norm[b]), xn_hl, sumsq, dm);
            ctx->launches++;
            EpiParams sw = base;
            sw.act_planes = act_hl; sw.ffn = d.ffn;
            ST((launch_gemm_tc<EPI_SWIGLU, float, NB>(ctx, GemmSite{nullptr, 2 * d.ffn, dm, nullptr, &ctx->tm_wgu[b], &ctx->tm_xn_big}, sw, nullptr, n_prob)));
            ST((launch_gemm_tc<EPI_RESID, float, NB>(ctx, GemmSite{nullptr, dm, d.ffn, nullptr, &ctx->tm_wdown[b], &ctx->tm_act_big}, resid, nullptr, n_prob)));
        }
    }
    match_rows_kernel<<<ceil_div(C, 128), 128, 0, ctx->stream>>>(pred, truth_dev, gamma, C, kptr<int>(ctx, ctx->kl.score_out));
    ctx->launches++;
    CU(cudaGetLastError());
    return SWIFT_OK;
}

double forward_bytes(const swift_ctx* ctx, const uint8_t* skip, int n_rows, int n_context, int kv_elem_bytes = 2)
{
    const swift_model_desc& d = ctx->d;
    const double es = (double)ctx->esize, kes = kv_elem_bytes > 0 ? (double)kv_elem_bytes : (double)kv_esize_of(&ctx->d);
    const double dm = d.d_model, qd = (double)d.n_heads * d.head_dim, kd = (double)d.n_kv_heads * d.head_dim;
    const double attn_w = (qd + 2 * kd) * dm + dm * qd, mlp_w = 3.0 * d.ffn * dm;
    double bytes = (double)d.vocab * dm * es;                      // output head
    for (int b = 0; b < d.n_blocks; ++b) {
        if (!(skip && skip[2 * b])) bytes += attn_w * es + 2.0 * kd * n_context * kes + 2.0 * kd * n_rows * kes;
        if (!(skip && skip[2 * b + 1])) bytes += mlp_w * es;
    }
    bytes += n_rows * (dm * es + (double)d.vocab * 4.0);           // embedding rows in, logits out
    return bytes;
}

} // namespace

// =============================================================================== tensor maps
namespace {

template <typename T, int MR>
cudaError_t set_attrs_mr()
{
    cudaError_t e = cudaFuncSetAttribute(gemm_simt_kernel<T, MR>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 1024 * 4);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_split_kernel<T, MR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(2 * ATTN_CHUNK * 256 * sizeof(T) + (MR * 256 + 3 * MR * ATTN_CHUNK) * 4));
    return e;
}
template <typename T>
cudaError_t set_attrs()
{
    cudaError_t e = cudaFuncSetAttribute(attn_split_kernel<T, 12>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(2 * ATTN_CHUNK * 256 * sizeof(T) + (12 * 256 + 3 * 12 * ATTN_CHUNK) * 4));
    if (e == cudaSuccess) e = set_attrs_mr<T, 1>();
    if (e == cudaSuccess) e = set_attrs_mr<T, 2>();
    if (e == cudaSuccess) e = set_attrs_mr<T, 4>();
    if (e == cudaSuccess) e = set_attrs_mr<T, 8>();
    if (e == cudaSuccess) e = set_attrs_mr<T, 16>();
    return e;
}
// Opt-in shared-memory sizes of every kernel, set once per device before anything is captured.
cudaError_t init_kernel_attrs()
{
    cudaError_t e = set_attrs<float>();
    if (e == cudaSuccess) e = set_attrs<__nv_bfloat16>();
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_PLAIN, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV, __nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    constexpr int big_smem = TcShape<TC_NB_MAX>::SMEM_BYTES;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_PLAIN, float, TC_NB_MAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, big_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID, float, TC_NB_MAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, big_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU, float, TC_NB_MAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, big_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV, float, TC_NB_MAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, big_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV, __nv_bfloat16, TC_NB_MAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, big_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_tile_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_tile_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM_BYTES);
    const int am_max = (int)attn_mma_smem_bytes(2, 262144 / ATTN_CHUNK);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_mma_kernel<float, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, am_max);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_mma_kernel<float, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, am_max);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_mma_kernel<__nv_bfloat16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, am_max);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_mma_kernel<__nv_bfloat16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, am_max);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(vocab_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VOCAB_CACHE_MAX_BYTES);
    return e;
}

// bf16 row-major [rows][cols] matrix, box = box_rows x 64 columns (128 bytes), 128-byte swizzle.
swift_status make_map(swift_ctx* ctx, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        CU(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !fn) return fail(ctx, SWIFT_ECUDA, "cuTensorMapEncodeTiled not available from the driver");
        encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, SWIFT_ECUDA, "cuTensorMapEncodeTiled failed with code %d (rows %llu, cols %llu)", (int)r,
                                       (unsigned long long)rows, (unsigned long long)cols);
    return SWIFT_OK;
}

swift_status make_all_maps(swift_ctx* ctx)
{
    const swift_model_desc& d = ctx->d;
    const uint64_t dm = d.d_model, qd = (uint64_t)d.n_heads * d.head_dim, kd = (uint64_t)d.n_kv_heads * d.head_dim;
    ctx->tm_wqkv.resize(d.n_blocks); ctx->tm_wo.resize(d.n_blocks); ctx->tm_wgu.resize(d.n_blocks); ctx->tm_wdown.resize(d.n_blocks);
    for (int b = 0; b < d.n_blocks; ++b) {
        ST(make_map(ctx, &ctx->tm_wqkv[b], ctx->wbase + ctx->wl.wqkv[b], qd + 2 * kd, dm, TC_TILE_N));
        ST(make_map(ctx, &ctx->tm_wo[b], ctx->wbase + ctx->wl.wo[b], dm, qd, TC_TILE_N));
        ST(make_map(ctx, &ctx->tm_wgu[b], ctx->wbase + ctx->wl.wgu[b], 2 * (uint64_t)d.ffn, dm, TC_TILE_N));
        ST(make_map(ctx, &ctx->tm_wdown[b], ctx->wbase + ctx->wl.wdown[b], dm, d.ffn, TC_TILE_N));
    }
    ST(make_map(ctx, &ctx->tm_lm_head, ctx->wbase + ctx->wl.lm_head, d.vocab, dm, TC_TILE_N));
    ST(make_map(ctx, &ctx->tm_embed, ctx->wbase + ctx->wl.embed, d.vocab, dm, TC_TILE_N));
    ST(make_map(ctx, &ctx->tm_xn, ctx->ws + ctx->kl.xn_hl, 2 * ROWS, dm, TC_COLS));
    ST(make_map(ctx, &ctx->tm_xa, ctx->ws + ctx->kl.xa_hl, 2 * ROWS, qd, TC_COLS));
    ST(make_map(ctx, &ctx->tm_act, ctx->ws + ctx->kl.act_hl, 2 * ROWS, d.ffn, TC_COLS));
    if (big_rows_of(&d) == (size_t)TC_BIG_ROWS) {
        ST(make_map(ctx, &ctx->tm_xn_big, ctx->ws + ctx->kl.xn_hl, 2 * TC_BIG_ROWS, dm, TcShape<TC_NB_MAX>::COLS));
        ST(make_map(ctx, &ctx->tm_xa_big, ctx->ws + ctx->kl.xa_hl, 2 * TC_BIG_ROWS, qd, TcShape<TC_NB_MAX>::COLS));
        ST(make_map(ctx, &ctx->tm_act_big, ctx->ws + ctx->kl.act_hl, 2 * TC_BIG_ROWS, d.ffn, TcShape<TC_NB_MAX>::COLS));
    }
    return SWIFT_OK;
}

} // namespace

// =============================================================================== C boundary
extern "C" {

size_t swift_weights_bytes(const swift_model_desc* d) { return desc_ok(d, nullptr) ? weight_layout(d).total : 0; }

size_t swift_kv_bytes(const swift_model_desc* d)
{
    if (!desc_ok(d, nullptr)) return 0;
    return (size_t)(d->max_positions / d->page_size + scratch_pages(d)) * page_bytes(d);
}

size_t swift_workspace_bytes(const swift_model_desc* d) { return desc_ok(d, nullptr) ? work_layout(d).total : 0; }

const char* swift_last_error(const swift_ctx* ctx) { return ctx ? ctx->err.c_str() : g_load_error.c_str(); }

swift_status swift_load(const swift_model_desc* desc, swift_devbuf weights, swift_devbuf kv_pool, swift_devbuf workspace,
                        void* cuda_stream, swift_ctx** out)
{
    swift_ctx* ctx = nullptr;   // for the error macros: errors before creation go to the thread-local text
    if (!out) return fail(nullptr, SWIFT_EINVAL, "out is null");
    *out = nullptr;
    std::string why;
    if (!desc_ok(desc, &why)) return fail(nullptr, SWIFT_EINVAL, "invalid model description: %s", why.c_str());
    if (!weights.dptr || !kv_pool.dptr || !workspace.dptr) return fail(nullptr, SWIFT_EINVAL, "null device buffer");
    if (((uintptr_t)weights.dptr | (uintptr_t)kv_pool.dptr | (uintptr_t)workspace.dptr) % ALIGN)
        return fail(nullptr, SWIFT_EINVAL, "device buffers must be 256-byte aligned");
    if (weights.bytes < swift_weights_bytes(desc) || kv_pool.bytes < swift_kv_bytes(desc) ||
        workspace.bytes < swift_workspace_bytes(desc))
        return fail(nullptr, SWIFT_ECAPACITY, "a device buffer is smaller than the size query says");
    int dev = 0, major = 0;
    CU(cudaGetDevice(&dev));
    CU(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major < 10) return fail(nullptr, SWIFT_EUNSUPPORTED, "this library is built for sm_100a only (device has major %d)", major);

    swift_ctx* c = new swift_ctx();
    c->d = *desc;
    c->stream = (cudaStream_t)cuda_stream;
    c->device = dev;
    c->esize = esize_of(desc);
    c->wbase = (char*)weights.dptr; c->kvbase = (char*)kv_pool.dptr; c->ws = (char*)workspace.dptr;
    c->wl = weight_layout(desc);
    c->kl = work_layout(desc);
    int shift = 0;
    while ((1 << shift) < desc->page_size) ++shift;
    c->kv = KvLayout{desc->n_blocks, desc->n_kv_heads, desc->head_dim, desc->page_size, shift};
    c->n_pages_main = desc->max_positions / desc->page_size;
    c->n_pages_scratch = scratch_pages(desc);
    c->max_splits = ceil_div(desc->max_positions, ATTN_CHUNK);
    c->phase = PH_LOADED; c->n = 0; c->pending = 0; c->n_prompt = 0; c->round = 0; c->last_k = 0; c->last_max_k = 0;
    c->round_open = false;
    c->mode = SWIFT_GREEDY; c->temperature = 1.f; c->top_p = 1.f; c->greedy_draft = false; c->seed = 0; c->engine = nullptr; c->tree_rows = 0; memset(&c->last_state, 0, sizeof(DevState)); c->launches = 0; c->h2d_bytes = 0; c->d2h_bytes = 0;
    ctx = c;
    c->use_tc = false;
    if (desc->dtype == SWIFT_BF16) {
        const swift_status ms = make_all_maps(c);
        if (ms != SWIFT_OK) { g_load_error = c->err; delete c; return ms; }   // (graphs not allocated yet)
        c->use_tc = true;
    }
    for (auto& e : c->ev) e = nullptr;
    c->use_graphs = getenv("SWIFT_NO_GRAPHS") == nullptr;
    {
        const char* e = getenv("SWIFT_ATTN_ROWS");           // rows per attention CTA: 1, 2, 4, 6, 8, 12 or 16
        const int v = e ? atoi(e) : 16;
        c->attn_rows_per_cta = (v == 1 || v == 2 || v == 4 || v == 6 || v == 8 || v == 12) ? v : 16;
    }
    c->fuse_combine = getenv("SWIFT_NO_FUSE_COMBINE") == nullptr;
    {
        // Tensor-core attention for the target model's decode forwards (verification, vanilla steps): opt-in with
        // SWIFT_ATTN_MMA=1.  Measured on the same box it lost to the streaming kernel at every shape tried (13B widths:
        // verification 0.648 against 0.662 of the roofline, vanilla steps 0.747 against 0.779); prefill chunks of many
        // rows always use it.
        const char* e = getenv("SWIFT_ATTN_MMA");
        c->attn_mma = e != nullptr && atoi(e) != 0;
    }
    c->prefetch_next = getenv("SWIFT_NO_PREFETCH_NEXT") == nullptr;
    {
        const char* e = getenv("SWIFT_PREFETCH_TILES");      // 16 KB tiles of the next GEMM each CTA asks L2 for
        c->prefetch_tiles = e ? std::max(0, std::min(256, atoi(e))) : 16;
    }
    // Programmatic dependent launch.  On by default for the tensor-core GEMM launches only: a GEMM's CTAs then start during
    // the tail of whatever precedes them and have their barriers, descriptors and first weight tile under way when its
    // results become visible (+1.6 to 1.9 % on whole 13B forwards).  As the secondary of such an edge the attention and
    // split-merge launches lose (their early CTAs sit beside the running GEMM), so SWIFT_PDL=1 (every launch) stays opt-in.
    c->pdl_next = false;
    c->pdl_gemms = getenv("SWIFT_NO_PDL_GEMMS") == nullptr;
    c->use_pdl = getenv("SWIFT_PDL") != nullptr;
    c->fuse = getenv("SWIFT_NO_FUSE") == nullptr && desc->head_dim <= TC_TILE_N;
    // prefill in chunks of up to TC_ROWS_MAX rows (SWIFT_NO_BIG_CHUNKS: 16 rows at a time, as decoding does)
    c->big_chunks = c->use_tc && c->fuse && big_rows_of(desc) == (size_t)TC_BIG_ROWS && getenv("SWIFT_NO_BIG_CHUNKS") == nullptr;
    c->whole_tiles = getenv("SWIFT_NO_WHOLE_TILES") == nullptr;
    {   // chunks of 512 rows: four 128-row problems per GEMM launch (SWIFT_MANY_PROBLEMS=1..4 for measurement)
        const char* e = getenv("SWIFT_MANY_PROBLEMS");
        c->many_problems = e ? std::max(1, std::min((int)TC_PROBS_MAX, atoi(e))) : (int)TC_PROBS_MAX;
    }
    c->attn_tile = getenv("SWIFT_NO_ATTN_TILE") == nullptr;      // chunks of many rows: 64-row query tiles with K,V staged in shared memory
    // Grouped-query models: the target model's decoding forwards (verification, vanilla steps) take that kernel too, one
    // CTA serving all query heads of a KV group, so that a K,V chunk is fetched and converted once per group
    c->attn_tile_decode = c->attn_tile && desc->head_dim == 128 &&
                          (desc->n_heads / desc->n_kv_heads >= 4 || getenv("SWIFT_ATTN_TILE_DECODE") != nullptr) &&
                          getenv("SWIFT_NO_ATTN_TILE_DECODE") == nullptr;
    c->attn_tile_drafts = getenv("SWIFT_NO_ATTN_TILE_DRAFTS") == nullptr;   // and so do its layer-skipped forwards (70B shape: +2 %)
    c->batched_scoring = c->big_chunks && getenv("SWIFT_NO_BATCHED_SCORING") == nullptr;
    c->graphs = new std::vector<FwdGraph>();
    c->graph_clock = 0;
    cudaError_t e = init_kernel_attrs();
    for (auto& ev : c->ev) if (e == cudaSuccess) e = cudaEventCreate(&ev);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws, 0, c->kl.total, c->stream);
    if (e == cudaSuccess) {
        const int half = desc->head_dim / 2, total = desc->max_positions * half;
        rope_table_kernel<<<ceil_div(total, 256), 256, 0, c->stream>>>(kptr<float2>(c, c->kl.rope), desc->max_positions, half,
                                                                     (double)desc->rope_theta);
        c->launches++;
        std::vector<int> pt(c->n_pages_main);
        for (int i = 0; i < c->n_pages_main; ++i) pt[i] = i;
        e = cudaMemcpyAsync(kptr<int>(c, c->kl.pt_main), pt.data(), pt.size() * 4, cudaMemcpyHostToDevice, c->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(kptr<int>(c, c->kl.pt_score), pt.data(), pt.size() * 4, cudaMemcpyHostToDevice, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        fail(nullptr, SWIFT_ECUDA, "set-up failed: %s", cudaGetErrorString(e));
        for (auto& ev : c->ev) if (ev) cudaEventDestroy(ev);
        delete c->graphs;
        delete c;
        return SWIFT_ECUDA;
    }
    *out = c;
    return SWIFT_OK;
}

swift_status swift_free(swift_ctx* ctx)
{
    if (!ctx) return SWIFT_OK;
    cudaStreamSynchronize(ctx->stream);
    for (auto& ev : ctx->ev) if (ev) cudaEventDestroy(ev);
    for (auto& g : *ctx->graphs) cudaGraphExecDestroy(g.exec);
    delete ctx->graphs;
    delete ctx->engine;
    delete ctx;
    return SWIFT_OK;
}

swift_status swift_pack_tensor(swift_ctx* ctx, swift_tensor_kind kind, int32_t block, const void* src, size_t src_bytes)
{
    if (!ctx || !src) return fail(ctx, SWIFT_EINVAL, "null argument");
    const swift_model_desc& d = ctx->d;
    const size_t es = ctx->esize, dm = d.d_model, qd = (size_t)d.n_heads * d.head_dim, kd = (size_t)d.n_kv_heads * d.head_dim;
    const bool per_block = kind >= SWIFT_T_WQ;
    if (per_block && (block < 0 || block >= d.n_blocks)) return fail(ctx, SWIFT_EINVAL, "block %d out of range", block);
    size_t dst = 0, bytes = 0;
    bool interleave = false;
    switch (kind) {
    case SWIFT_T_EMBED: dst = ctx->wl.embed; bytes = (size_t)d.vocab * dm * es; break;
    case SWIFT_T_LM_HEAD: dst = ctx->wl.lm_head; bytes = (size_t)d.vocab * dm * es; break;
    case SWIFT_T_FINAL_NORM: dst = ctx->wl.final_norm; bytes = dm * 4; break;
    case SWIFT_T_WQ: dst = ctx->wl.wqkv[block]; bytes = qd * dm * es; break;
    case SWIFT_T_WK: dst = ctx->wl.wqkv[block] + qd * dm * es; bytes = kd * dm * es; break;
    case SWIFT_T_WV: dst = ctx->wl.wqkv[block] + (qd + kd) * dm * es; bytes = kd * dm * es; break;
    case SWIFT_T_WO: dst = ctx->wl.wo[block]; bytes = dm * qd * es; break;
    case SWIFT_T_WGATE: dst = ctx->wl.wgu[block]; bytes = (size_t)d.ffn * dm * es; interleave = true; break;
    case SWIFT_T_WUP: dst = ctx->wl.wgu[block] + 16 * dm * es; bytes = (size_t)d.ffn * dm * es; interleave = true; break;
    case SWIFT_T_WDOWN: dst = ctx->wl.wdown[block]; bytes = dm * (size_t)d.ffn * es; break;
    case SWIFT_T_ATTN_NORM: dst = ctx->wl.attn_norm[block]; bytes = dm * 4; break;
    case SWIFT_T_MLP_NORM: dst = ctx->wl.mlp_norm[block]; bytes = dm * 4; break;
    default: return fail(ctx, SWIFT_EINVAL, "unknown tensor kind %d", (int)kind);
    }
    if (src_bytes != bytes) return fail(ctx, SWIFT_EINVAL, "tensor kind %d expects %zu bytes, got %zu", (int)kind, bytes, src_bytes);
    CU(cudaStreamSynchronize(ctx->stream));
    if (interleave) {
        const size_t group = 16 * dm * es;       // 16 rows of gate (or up) ...
        CU(cudaMemcpy2D(ctx->wbase + dst, 2 * group, src, group, group, d.ffn / 16, cudaMemcpyHostToDevice));  // ... every 32 rows
    } else {
        CU(cudaMemcpy(ctx->wbase + dst, src, bytes, cudaMemcpyHostToDevice));
    }
    return SWIFT_OK;
}

swift_status swift_set_sampling(swift_ctx* ctx, int32_t mode, float temperature, uint64_t seed)
{
    if (!ctx) return SWIFT_EINVAL;
    if (mode != SWIFT_GREEDY && mode != SWIFT_SAMPLING) return fail(ctx, SWIFT_EINVAL, "mode must be SWIFT_GREEDY or SWIFT_SAMPLING");
    if (!(temperature > 0.f)) return fail(ctx, SWIFT_EINVAL, "temperature must be positive");
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "cannot change the acceptance strategy inside a round");
    ctx->mode = mode; ctx->temperature = temperature; ctx->seed = seed;
    return SWIFT_OK;
}

swift_status swift_set_greedy_draft(swift_ctx* ctx, int32_t on)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "cannot change the drafting rule inside a round");
    ctx->greedy_draft = on != 0;
    return SWIFT_OK;
}

swift_status swift_set_top_p(swift_ctx* ctx, float top_p)
{
    if (!ctx) return SWIFT_EINVAL;
    if (!(top_p > 0.f) || top_p > 1.f) return fail(ctx, SWIFT_EINVAL, "top_p must be in (0, 1]");
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "cannot change the sampling distribution inside a round");
    ctx->top_p = top_p;
    return SWIFT_OK;
}

swift_status swift_forward_rows(swift_ctx* ctx, const int32_t* tokens, int32_t n_rows, int32_t pos0, const uint8_t* skip,
                                int32_t write_kv, float* logits_host, int32_t* argmax_host)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "a round is open");
    if (n_rows < 1 || pos0 < 0) return fail(ctx, SWIFT_EINVAL, "n_rows >= 1 and pos0 >= 0 required");
    if (pos0 > ctx->n) return fail(ctx, SWIFT_EINVAL, "pos0 %d beyond the committed length %d", pos0, ctx->n);
    if (pos0 + n_rows > ctx->d.max_positions) return fail(ctx, SWIFT_ECAPACITY, "rows run past max_positions");
    if (!write_kv && n_rows > MAX_SCORE_ROWS) return fail(ctx, SWIFT_ECAPACITY, "at most %d rows without KV write", MAX_SCORE_ROWS);
    ST(check_tokens(ctx, tokens, n_rows));
    const int* pt = pt_main(ctx);
    if (!write_kv) { ST(prepare_scratch(ctx, pos0, pos0 + n_rows)); pt = pt_score(ctx); }
    ST(run_rows(ctx, tokens, n_rows, pos0, skip, pt, (logits_host || argmax_host) ? 2 : 0, logits_host, argmax_host, nullptr));
    DevState hs;
    return read_state(ctx, &hs);
}

swift_status swift_prefill(swift_ctx* ctx, const int32_t* tokens, int32_t n, int32_t* first_token)
{
    if (!ctx) return SWIFT_EINVAL;
    if (n < 1) return fail(ctx, SWIFT_EINVAL, "prompt must have at least one token");
    if (n + 1 > ctx->d.max_positions) return fail(ctx, SWIFT_ECAPACITY, "prompt of %d tokens exceeds max_positions %d", n, ctx->d.max_positions);
    ST(check_tokens(ctx, tokens, n));
    ctx->round_open = false;
    ctx->n = 0;
    int last_rows = 0;
    // All but the last (up to 16) rows go through in chunks of up to TC_BIG_ROWS rows where that path exists: every weight
    // is then streamed once per 128 rows instead of once per 16.  The last rows take the decoding path, which ends in
    // the output head.
    int done = 0;
    if (ctx->big_chunks && n > 2 * ROWS) {
        const int big_total = ((n - 1) / ROWS) * ROWS;           // leaves 1..16 rows
        DevState* st = state_of(ctx);
        const int chunk = ctx->many_problems * TC_ROWS_MAX;
        for (int c0 = 0; c0 < big_total; c0 += chunk) {
            const int rows = std::min(chunk, big_total - c0);
            CU(copy_async(ctx, kptr<int>(ctx, ctx->kl.big_tok), tokens + c0, (size_t)rows * 4, cudaMemcpyHostToDevice));
            set_rows_kernel<<<1, 1, 0, ctx->stream>>>(st, c0, rows);
            ctx->launches++;
            if (ctx->d.kv_dtype == SWIFT_BF16) ST(forward_chunk_big<__nv_bfloat16>(ctx, rows, pt_main(ctx)));
            else ST(forward_chunk_big<float>(ctx, rows, pt_main(ctx)));
        }
        done = big_total;
    }
    ST(run_rows(ctx, tokens + done, n - done, done, nullptr, pt_main(ctx), 1, nullptr, nullptr, &last_rows));
    if (ctx->mode == SWIFT_SAMPLING) {
        sample_row_kernel<<<1, VOCAB_THREADS, 0, ctx->stream>>>(state_of(ctx), kptr<float>(ctx, ctx->kl.logits), ctx->d.vocab,
                                                                last_rows - 1, 1.0f / ctx->temperature, ctx->seed, 0u, 0u);
        ctx->launches++;
    }
    DevState hs;
    swift_status s = read_state(ctx, &hs);
    if (s != SWIFT_OK) { ctx->phase = PH_LOADED; return s; }
    const int tok = ctx->mode == SWIFT_SAMPLING ? hs.next_token : hs.argmax[last_rows - 1];
    ctx->n = n; ctx->n_prompt = n; ctx->pending = tok; ctx->round = 0;
    ctx->hist.assign(tokens, tokens + n);
    ctx->hist.push_back(tok);
    ctx->phase = PH_READY;
    if (first_token) *first_token = tok;
    return SWIFT_OK;
}

swift_status swift_set_pending(swift_ctx* ctx, int32_t token, int32_t rounds_done)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->phase != PH_READY) return fail(ctx, SWIFT_ESTATE, "swift_set_pending needs a prefilled context with no open round");
    if (token < 0 || token >= ctx->d.vocab) return fail(ctx, SWIFT_EINVAL, "token id %d outside [0, %d)", token, ctx->d.vocab);
    ctx->pending = token;
    ctx->hist.back() = token;
    if (rounds_done >= 0) ctx->round = rounds_done;
    return SWIFT_OK;
}

swift_status swift_draft(swift_ctx* ctx, const uint8_t* skip, int32_t max_k, float stop_conf, int32_t* tokens_host,
                         float* conf_host, int32_t* k_host)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->phase != PH_READY) return fail(ctx, SWIFT_ESTATE, "swift_draft needs a prefilled context with no open round");
    if (!skip) return fail(ctx, SWIFT_EINVAL, "skip_mask is null");
    if (max_k < 0 || max_k > ctx->d.max_draft) return fail(ctx, SWIFT_ECAPACITY, "max_k %d outside 0..max_draft (%d)", max_k, ctx->d.max_draft);
    if (ctx->n + max_k + 1 > ctx->d.max_positions) return fail(ctx, SWIFT_ECAPACITY, "KV cache too small for %d more positions", max_k + 1);
    ST(enqueue_draft(ctx, skip, max_k, stop_conf));
    DevState hs;
    ST(read_state(ctx, &hs));
    ctx->last_k = hs.n_drafted;
    ctx->phase = PH_DRAFTED;
    for (int j = 0; j < hs.n_drafted; ++j) {
        if (tokens_host) tokens_host[j] = hs.draft_tok[j + 1];
        if (conf_host) conf_host[j] = hs.conf[j];
    }
    if (k_host) *k_host = hs.n_drafted;
    return SWIFT_OK;
}

swift_status swift_verify(swift_ctx* ctx, const int32_t* tokens_host, int32_t k, int32_t* target_argmax, float* logits_host)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->phase != PH_READY && ctx->phase != PH_DRAFTED) return fail(ctx, SWIFT_ESTATE, "swift_verify needs a prefilled context");
    int rows_launch, forced_k;
    if (tokens_host) {
        if (k < 0 || k > SWIFT_MAX_ROWS - 1) return fail(ctx, SWIFT_ECAPACITY, "k %d outside 0..%d", k, SWIFT_MAX_ROWS - 1);
        if (ctx->mode == SWIFT_SAMPLING && k > 0 && ctx->phase != PH_DRAFTED)
            return fail(ctx, SWIFT_ESTATE, "sampling acceptance needs the draft distributions of swift_draft");
        // acceptance compares p_j with the distribution q_j kept from draft step j: there are only last_k of those
        if (ctx->mode == SWIFT_SAMPLING && k > ctx->last_k)
            return fail(ctx, SWIFT_ECAPACITY, "sampling acceptance of %d tokens, but swift_draft produced %d draft distributions", k, ctx->last_k);
        if (k > 0) ST(check_tokens(ctx, tokens_host, k));
        if (ctx->n + k + 1 > ctx->d.max_positions) return fail(ctx, SWIFT_ECAPACITY, "KV cache too small");
        if (ctx->phase == PH_READY) {
            ctx->round++;
            launch_begin_round(ctx, 0.f);
            ctx->round_open = true;
        }
        if (k > 0) CU(copy_async(ctx, state_of(ctx)->draft_tok + 1, tokens_host, k * 4, cudaMemcpyHostToDevice));
        rows_launch = k + 1; forced_k = k;
    } else {
        if (ctx->phase != PH_DRAFTED) return fail(ctx, SWIFT_ESTATE, "no draft to verify: call swift_draft or pass tokens");
        rows_launch = ctx->last_k + 1; forced_k = -1;
        if (tree_active(ctx) && ctx->n + std::max(ctx->tree_rows, rows_launch) > ctx->d.max_positions)
            return fail(ctx, SWIFT_ECAPACITY, "KV cache too small for the rows of the token tree");
    }
    ST(enqueue_verify(ctx, rows_launch, forced_k));
    DevState hs;
    ST(read_state(ctx, &hs));
    ctx->last_k = hs.n_drafted;
    ctx->phase = PH_VERIFIED;
    const int rows = hs.tree_rows > 0 ? hs.tree_rows : hs.n_drafted + 1;
    if (target_argmax) for (int r = 0; r < rows; ++r) target_argmax[r] = hs.argmax[r];
    if (logits_host) {
        CU(copy_async(ctx, logits_host, kptr<float>(ctx, ctx->kl.logits), (size_t)rows * ctx->d.vocab * 4, cudaMemcpyDeviceToHost));
        CU(cudaStreamSynchronize(ctx->stream));
    }
    return SWIFT_OK;
}

swift_status swift_set_tree(swift_ctx* ctx, int32_t tree_rows)
{
    if (!ctx) return SWIFT_EINVAL;
    if (tree_rows != 0 && (tree_rows < 2 || tree_rows > SWIFT_MAX_ROWS)) return fail(ctx, SWIFT_EINVAL, "tree_rows must be 0 or in 2..%d", SWIFT_MAX_ROWS);
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "cannot change the verification form inside a round");
    ctx->tree_rows = tree_rows;
    return SWIFT_OK;
}

swift_status swift_verify_tree(swift_ctx* ctx, const int32_t* tokens_host, const int32_t* parent_host, int32_t n_rows,
                               int32_t* target_argmax, float* logits_host)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->phase != PH_READY && ctx->phase != PH_DRAFTED) return fail(ctx, SWIFT_ESTATE, "swift_verify_tree needs a prefilled context");
    if (ctx->mode != SWIFT_GREEDY) return fail(ctx, SWIFT_EUNSUPPORTED, "token trees are verified under greedy decoding only");
    if (!tokens_host || !parent_host) return fail(ctx, SWIFT_EINVAL, "null argument");
    if (n_rows < 1 || n_rows > SWIFT_MAX_ROWS) return fail(ctx, SWIFT_ECAPACITY, "a tree of %d rows; at most %d", n_rows, SWIFT_MAX_ROWS);
    if (tokens_host[0] != ctx->pending) return fail(ctx, SWIFT_EINVAL, "row 0 of the tree must be the pending token");
    if (parent_host[0] != -1) return fail(ctx, SWIFT_EINVAL, "row 0 is the root: its parent must be -1");
    for (int i = 1; i < n_rows; ++i)
        if (parent_host[i] < 0 || parent_host[i] >= i) return fail(ctx, SWIFT_EINVAL, "parent of row %d must be an earlier row", i);
    ST(check_tokens(ctx, tokens_host, n_rows));
    if (ctx->n + n_rows > ctx->d.max_positions) return fail(ctx, SWIFT_ECAPACITY, "KV cache too small");
    if (ctx->phase == PH_READY) {
        ctx->round++;
        launch_begin_round(ctx, 0.f);
        ctx->round_open = true;
    }
    DevState* st = state_of(ctx);
    CU(copy_async(ctx, st->draft_tok, tokens_host, (size_t)n_rows * 4, cudaMemcpyHostToDevice));
    CU(copy_async(ctx, st->row_parent, parent_host, (size_t)n_rows * 4, cudaMemcpyHostToDevice));
    begin_verify_given_tree_kernel<<<1, 1, 0, ctx->stream>>>(st, ctx->n, n_rows);
    ctx->launches++;
    HeadOpts head;
    head.run = true;
    ctx->tree_forward = true;
    const swift_status fs = forward_cached(ctx, n_rows, st->draft_tok, nullptr, pt_main(ctx), head);
    ctx->tree_forward = false;
    ST(fs);
    DevState hs;
    ST(read_state(ctx, &hs));
    ctx->last_k = hs.n_drafted;
    ctx->phase = PH_VERIFIED;
    if (target_argmax) for (int r = 0; r < n_rows; ++r) target_argmax[r] = hs.argmax[r];
    if (logits_host) {
        CU(copy_async(ctx, logits_host, kptr<float>(ctx, ctx->kl.logits), (size_t)n_rows * ctx->d.vocab * 4, cudaMemcpyDeviceToHost));
        CU(cudaStreamSynchronize(ctx->stream));
    }
    return SWIFT_OK;
}

int32_t swift_tree_rows(const swift_ctx* ctx, int32_t* tokens_host, int32_t* parent_host, int32_t* depth_host)
{
    if (!ctx) return -1;
    const DevState& hs = ctx->last_state;
    const int rows = hs.tree_rows > 0 ? hs.tree_rows : 0;
    for (int r = 0; r < rows; ++r) {
        if (tokens_host) tokens_host[r] = hs.draft_tok[r];
        if (parent_host) parent_host[r] = hs.row_parent[r];
        if (depth_host) depth_host[r] = hs.row_depth[r];
    }
    return rows;
}

swift_status swift_accept(swift_ctx* ctx, int32_t* n_accepted, int32_t* next_token)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->phase != PH_VERIFIED) return fail(ctx, SWIFT_ESTATE, "swift_accept needs a verified round");
    ST(enqueue_accept(ctx));
    DevState hs;
    ST(read_state(ctx, &hs));
    commit_round(ctx, hs);
    if (n_accepted) *n_accepted = hs.n_accepted;
    if (next_token) *next_token = hs.next_token;
    return SWIFT_OK;
}

swift_status swift_score_skipsets(swift_ctx* ctx, const uint8_t* masks, int32_t C, int32_t gamma, float* matchness)
{
    if (!ctx) return SWIFT_EINVAL;
    if (ctx->phase != PH_READY) return fail(ctx, SWIFT_ESTATE, "swift_score_skipsets needs a prefilled context with no open round");
    if (!masks || !matchness) return fail(ctx, SWIFT_EINVAL, "null argument");
    if (C < 1 || C > 1024) return fail(ctx, SWIFT_ECAPACITY, "C must be in 1..1024");
    if (gamma < 1 || gamma > MAX_SCORE_ROWS) return fail(ctx, SWIFT_ECAPACITY, "gamma must be in 1..%d", MAX_SCORE_ROWS);
    if (gamma > ctx->n) return fail(ctx, SWIFT_EINVAL, "gamma %d exceeds the %d cached positions", gamma, ctx->n);
    ST(enqueue_score(ctx, masks, C, gamma));
    std::vector<int> counts(C);
    CU(copy_async(ctx, counts.data(), kptr<int>(ctx, ctx->kl.score_out), C * 4, cudaMemcpyDeviceToHost));
    DevState hs;
    ST(read_state(ctx, &hs));
    for (int c = 0; c < C; ++c) matchness[c] = (float)counts[c] / (float)gamma;
    return SWIFT_OK;
}

swift_status swift_gemm(swift_ctx* ctx, int32_t which, int32_t block, const float* x_host, int32_t n_rows, float* y_host)
{
    if (!ctx || !x_host || !y_host) return fail(ctx, SWIFT_EINVAL, "null argument");
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "a round is open");
    const swift_model_desc& d = ctx->d;
    if (which < 0 || which > 4 || n_rows < 1 || n_rows > TC_BIG_ROWS || block < 0 || block >= d.n_blocks)
        return fail(ctx, SWIFT_EINVAL, "bad which / block / n_rows");
    if (n_rows > ROWS && !(ctx->use_tc && ctx->big_chunks)) return fail(ctx, SWIFT_EUNSUPPORTED, "no many-row GEMM for this model or kernel choice");
    const int dm = d.d_model, qd = d.n_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim;
    const int N = which == 0 ? qd + 2 * kd : which == 1 ? dm : which == 2 ? 2 * d.ffn : which == 3 ? dm : d.vocab;
    const int K = which == 1 ? qd : which == 3 ? d.ffn : dm;
    float* X = which == 1 ? kptr<float>(ctx, ctx->kl.xa) : which == 3 ? kptr<float>(ctx, ctx->kl.act) : kptr<float>(ctx, ctx->kl.xn);
    const size_t woff = which == 0 ? ctx->wl.wqkv[block] : which == 1 ? ctx->wl.wo[block] : which == 2 ? ctx->wl.wgu[block]
                        : which == 3 ? ctx->wl.wdown[block] : ctx->wl.lm_head;
    if (n_rows > ROWS) {   // the many-row form (prefill chunks, side-by-side scoring), plain epilogue
        if (N > d.vocab) return fail(ctx, SWIFT_ECAPACITY, "output of %d columns does not fit the buffer used for this call", N);
        __nv_bfloat16* planes = which == 1 ? kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl) : which == 3 ? kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl)
                                           : kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
        for (int r0 = 0; r0 < n_rows; r0 += ROWS) {            // rows reach their planes 16 at a time through the 16-row buffer
            const int nr = std::min((int)ROWS, n_rows - r0);
            CU(copy_async(ctx, X, x_host + (size_t)r0 * K, (size_t)nr * K * 4, cudaMemcpyHostToDevice));
            split_planes_kernel<<<dim3(ceil_div(K, 256), nr), 256, 0, ctx->stream>>>(X, planes, K, r0);
            ctx->launches++;
        }
        set_rows_kernel<<<1, 1, 0, ctx->stream>>>(state_of(ctx), 0, n_rows);
        ctx->launches++;
        EpiParams ep;
        memset(&ep, 0, sizeof ep);
        ep.sum_rows = TC_BIG_ROWS;
        GemmSite g{nullptr, N, K, nullptr,
                   which == 0 ? &ctx->tm_wqkv[block] : which == 1 ? &ctx->tm_wo[block] : which == 2 ? &ctx->tm_wgu[block]
                   : which == 3 ? &ctx->tm_wdown[block] : &ctx->tm_lm_head,
                   which == 1 ? &ctx->tm_xa_big : which == 3 ? &ctx->tm_act_big : &ctx->tm_xn_big};
        float* Y = kptr<float>(ctx, ctx->kl.score_logits);
        ST(launch_gemm_tc_y<TC_NB_MAX>(ctx, g, ep, Y, ceil_div(n_rows, TC_ROWS_MAX)));
        CU(copy_async(ctx, y_host, Y, (size_t)n_rows * N * 4, cudaMemcpyDeviceToHost));
        DevState hs;
        return read_state(ctx, &hs);
    }
    CU(copy_async(ctx, X, x_host, (size_t)n_rows * K * 4, cudaMemcpyHostToDevice));
    set_rows_kernel<<<1, 1, 0, ctx->stream>>>(state_of(ctx), 0, n_rows);
    ctx->launches++;
    GemmSite g{X, N, K, ctx->wbase + woff, nullptr, nullptr};
    if (ctx->use_tc) {
        __nv_bfloat16* planes = which == 1 ? kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl) : which == 3 ? kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl)
                                           : kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
        split_planes_kernel<<<dim3(ceil_div(K, 256), n_rows), 256, 0, ctx->stream>>>(X, planes, K, 0);
        ctx->launches++;
        g.mapW = which == 0 ? &ctx->tm_wqkv[block] : which == 1 ? &ctx->tm_wo[block] : which == 2 ? &ctx->tm_wgu[block]
                 : which == 3 ? &ctx->tm_wdown[block] : &ctx->tm_lm_head;
        g.mapX = which == 1 ? &ctx->tm_xa : which == 3 ? &ctx->tm_act : &ctx->tm_xn;
    }
    int S = 0;
    if (d.dtype == SWIFT_BF16) ST(run_gemm<__nv_bfloat16>(ctx, mr_of(n_rows), g, &S));
    else ST(run_gemm<float>(ctx, mr_of(n_rows), g, &S));
    std::vector<float> slab((size_t)n_rows * N);
    std::fill(y_host, y_host + (size_t)n_rows * N, 0.f);
    for (int s = 0; s < S; ++s) {          // slabs are added in slab order, as the consumers on the device do
        CU(copy_async(ctx, slab.data(), kptr<float>(ctx, ctx->kl.part) + (size_t)s * ROWS * N, slab.size() * 4, cudaMemcpyDeviceToHost));
        CU(cudaStreamSynchronize(ctx->stream));
        for (size_t i = 0; i < slab.size(); ++i) y_host[i] += slab[i];
    }
    DevState hs;
    return read_state(ctx, &hs);
}

swift_status swift_many_row_schedule(int32_t N, int32_t K, int32_t* grid_host, int32_t* max_share_host)
{
    if (!grid_host || !max_share_host || N < 1 || K < 1) return SWIFT_EINVAL;
    const int grid = many_row_grid(N, K);
    *grid_host = grid;
    *max_share_host = max_segments(N, K, grid);
    return SWIFT_OK;
}

swift_status swift_probe_wait_limit(swift_ctx* ctx, int32_t limit_us)
{
    if (!ctx) return SWIFT_EINVAL;
    if (limit_us < 1 || limit_us > 100000) return fail(ctx, SWIFT_EINVAL, "limit_us must be in 1..100000");
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "a round is open");
    wait_probe_kernel<<<1, 32, 0, ctx->stream>>>(state_of(ctx), (long long)limit_us * 2000LL);   // about 2 cycles per nanosecond
    ctx->launches++;
    CU(cudaGetLastError());
    DevState hs;
    return read_state(ctx, &hs);
}

swift_status swift_set_gemm_impl(swift_ctx* ctx, int32_t impl)
{
    if (!ctx) return SWIFT_EINVAL;
    if (impl != 0 && impl != 1) return fail(ctx, SWIFT_EINVAL, "impl must be 0 (SIMT) or 1 (tensor cores)");
    if (impl == 1 && ctx->d.dtype != SWIFT_BF16) return fail(ctx, SWIFT_EUNSUPPORTED, "the tensor-core GEMM needs bf16 weights");
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "a round is open");
    ctx->use_tc = impl == 1;
    return SWIFT_OK;
}

int32_t swift_committed_length(const swift_ctx* ctx) { return ctx ? ctx->n : -1; }
int64_t swift_launch_count(const swift_ctx* ctx) { return ctx ? ctx->launches : -1; }
int32_t swift_final_skip_mask(const swift_ctx* ctx, uint8_t* mask_host)
{
    if (!ctx || ctx->last_mask.empty()) return -1;
    if (mask_host) memcpy(mask_host, ctx->last_mask.data(), ctx->last_mask.size());
    return (int32_t)ctx->last_mask.size();
}
int32_t swift_round_times(const swift_ctx* ctx, int32_t capacity, float* ms_draft, float* ms_verify, double* bytes_draft,
                          double* bytes_verify, int32_t* drafted)
{
    if (!ctx) return -1;
    const int n = (int)ctx->round_times.size();
    for (int i = 0; i < n && i < capacity; ++i) {
        const auto& r = ctx->round_times[i];
        if (ms_draft) ms_draft[i] = r.ms_draft;
        if (ms_verify) ms_verify[i] = r.ms_verify;
        if (bytes_draft) bytes_draft[i] = r.bytes_draft;
        if (bytes_verify) bytes_verify[i] = r.bytes_verify;
        if (drafted) drafted[i] = r.drafted;
    }
    return n;
}
int32_t swift_round_bytes_stored(const swift_ctx* ctx, int32_t capacity, double* bytes_draft, double* bytes_verify)
{
    if (!ctx) return -1;
    const int n = (int)ctx->round_times.size();
    for (int i = 0; i < n && i < capacity; ++i) {
        if (bytes_draft) bytes_draft[i] = ctx->round_times[i].stored_draft;
        if (bytes_verify) bytes_verify[i] = ctx->round_times[i].stored_verify;
    }
    return n;
}
double swift_forward_bytes(const swift_ctx* ctx, const uint8_t* skip, int32_t n_rows, int32_t n_context, int32_t kv_elem_bytes)
{
    return ctx ? forward_bytes(ctx, skip, n_rows, n_context, kv_elem_bytes) : 0.0;
}

} // extern "C"

// =============================================================================== proposal engine (host only)
struct swift_opt { swopt::LayerOpt impl; swift_opt(int nb, int m, int beta, uint64_t seed, int pool) : impl(nb, m, beta, seed, pool) {} };

namespace {
void blocks_to_mask(const swopt::BlockSet& s, int n_blocks, uint8_t* mask)
{
    memset(mask, 0, 2 * (size_t)n_blocks);
    for (int b : s) mask[2 * b] = mask[2 * b + 1] = 1;
}
swopt::BlockSet mask_to_blocks(const uint8_t* mask, int n_blocks)
{
    swopt::BlockSet s;
    for (int b = 0; b < n_blocks; ++b) if (mask[2 * b] && mask[2 * b + 1]) s.push_back(b);
    return s;
}
} // namespace

extern "C" {

swift_opt* swift_opt_create(int32_t n_blocks, int32_t n_skip_blocks, int32_t beta, uint64_t seed, int32_t pool)
{
    if (n_blocks < 2 || n_skip_blocks < 1 || n_skip_blocks >= n_blocks || beta < 0 || pool < 1) return nullptr;
    return new swift_opt(n_blocks, n_skip_blocks, beta, seed, pool);
}
void swift_opt_free(swift_opt* opt) { delete opt; }
swift_status swift_opt_suggest(swift_opt* opt, uint8_t* mask_host, int32_t* is_bayesian_host)
{
    if (!opt || !mask_host) return SWIFT_EINVAL;
    const bool bayes = opt->impl.beta > 0 && (opt->impl.step + 1) % opt->impl.beta == 0 && !opt->impl.X.empty();
    blocks_to_mask(opt->impl.suggest(), opt->impl.nb, mask_host);
    if (is_bayesian_host) *is_bayesian_host = bayes ? 1 : 0;
    return SWIFT_OK;
}
swift_status swift_opt_observe(swift_opt* opt, const uint8_t* mask_host, float matchness)
{
    if (!opt || !mask_host) return SWIFT_EINVAL;
    opt->impl.observe(mask_to_blocks(mask_host, opt->impl.nb), (double)matchness);
    return SWIFT_OK;
}

} // extern "C"

// =============================================================================== inspection, generate
extern "C" {

swift_status swift_read_kv(swift_ctx* ctx, int32_t block, int32_t which, int32_t pos0, int32_t count, float* out_host)
{
    if (!ctx || !out_host) return fail(ctx, SWIFT_EINVAL, "null argument");
    if (block < 0 || block >= ctx->d.n_blocks || (which != 0 && which != 1)) return fail(ctx, SWIFT_EINVAL, "bad block or which");
    if (pos0 < 0 || count < 1 || pos0 + count > ctx->d.max_positions) return fail(ctx, SWIFT_EINVAL, "bad position range");
    const size_t per_pos = (size_t)ctx->d.n_kv_heads * ctx->d.head_dim;
    const int step = (int)std::max<size_t>(1, std::min<size_t>(count, ctx->kl.part_floats / per_pos));
    float* stage = kptr<float>(ctx, ctx->kl.part);
    for (int c0 = 0; c0 < count; c0 += step) {
        const int cnt = std::min(step, count - c0);
        if (ctx->d.kv_dtype == SWIFT_BF16)
            kv_read_kernel<__nv_bfloat16><<<64, 256, 0, ctx->stream>>>(reinterpret_cast<const __nv_bfloat16*>(ctx->kvbase),
                                                                      pt_main(ctx), ctx->kv, block, which, pos0 + c0, cnt, stage);
        else
            kv_read_kernel<float><<<64, 256, 0, ctx->stream>>>(reinterpret_cast<const float*>(ctx->kvbase), pt_main(ctx),
                                                               ctx->kv, block, which, pos0 + c0, cnt, stage);
        ctx->launches++;
        CU(copy_async(ctx, out_host + (size_t)c0 * per_pos, stage, (size_t)cnt * per_pos * 4, cudaMemcpyDeviceToHost));
        CU(cudaStreamSynchronize(ctx->stream));
    }
    return SWIFT_OK;
}

} // extern "C"

template <typename T>
static swift_status time_gemm_t(swift_ctx* ctx, int which, int n_rows, int iters, float* ms, double* bytes)
{
    const swift_model_desc& d = ctx->d;
    const int dm = d.d_model, qd = d.n_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim;
    const int N = which == 0 ? qd + 2 * kd : which == 1 ? dm : which == 2 ? 2 * d.ffn : which == 3 ? dm : d.vocab;
    const int K = which == 1 ? qd : which == 3 ? d.ffn : dm;
    const float* X = which == 1 ? kptr<float>(ctx, ctx->kl.xa) : which == 3 ? kptr<float>(ctx, ctx->kl.act) : kptr<float>(ctx, ctx->kl.xn);
    set_rows_kernel<<<1, 1, 0, ctx->stream>>>(state_of(ctx), 0, n_rows);
    ctx->launches++;
    GemmPlan p;
    auto weight = [&](int i) -> const T* {
        const int b = i % d.n_blocks;
        switch (which) {
        case 0: return wptr<T>(ctx, ctx->wl.wqkv[b]);
        case 1: return wptr<T>(ctx, ctx->wl.wo[b]);
        case 2: return wptr<T>(ctx, ctx->wl.wgu[b]);
        case 3: return wptr<T>(ctx, ctx->wl.wdown[b]);
        default: return (i & 1) ? wptr<T>(ctx, ctx->wl.embed) : wptr<T>(ctx, ctx->wl.lm_head);
        }
    };
    auto site = [&](int i) -> GemmSite {
        const int b = i % d.n_blocks;
        const CUtensorMap* mw = nullptr;
        if (ctx->use_tc)
            mw = which == 0 ? &ctx->tm_wqkv[b] : which == 1 ? &ctx->tm_wo[b] : which == 2 ? &ctx->tm_wgu[b] : which == 3 ? &ctx->tm_wdown[b]
                 : (i & 1) ? &ctx->tm_embed : &ctx->tm_lm_head;
        const CUtensorMap* mx = which == 1 ? &ctx->tm_xa : which == 3 ? &ctx->tm_act : &ctx->tm_xn;
        return GemmSite{X, N, K, weight(i), mw, mx};
    };
    int S = 0;
    (void)p;
    if (n_rows > ROWS) {   // the many-row form (prefill chunks, side-by-side scoring): plain epilogue into the scoring logits buffer
        if (!ctx->big_chunks) return fail(ctx, SWIFT_EUNSUPPORTED, "no many-row GEMM for this model");
        if (N > d.vocab) return fail(ctx, SWIFT_ECAPACITY, "output of %d columns does not fit the buffer used for timing", N);
        EpiParams ep;
        memset(&ep, 0, sizeof ep);
        ep.sum_rows = TC_BIG_ROWS;
        {   // the planes this launch reads get defined, non-trivial contents first
            __nv_bfloat16* planes = which == 1 ? kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl) : which == 3 ? kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl)
                                               : kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
            fill_planes_kernel<<<296, 256, 0, ctx->stream>>>(planes, (size_t)2 * TC_BIG_ROWS * K);
            ctx->launches++;
        }
        auto big = [&](int i) -> swift_status {
            GemmSite g = site(i);
            g.mapX = which == 1 ? &ctx->tm_xa_big : which == 3 ? &ctx->tm_act_big : &ctx->tm_xn_big;
            return launch_gemm_tc_y<TC_NB_MAX>(ctx, g, ep, kptr<float>(ctx, ctx->kl.score_logits), ceil_div(n_rows, TC_ROWS_MAX));
        };
        for (int i = 0; i < 3; ++i) ST(big(i));
        CU(cudaEventRecord(ctx->ev[0], ctx->stream));
        for (int i = 0; i < iters; ++i) ST(big(i + 3));
        CU(cudaEventRecord(ctx->ev[1], ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
        float t = 0.f;
        CU(cudaEventElapsedTime(&t, ctx->ev[0], ctx->ev[1]));
        *ms = t / (float)iters;
        *bytes = (double)N * K * sizeof(T);
        DevState hs;
        return read_state(ctx, &hs);
    }
    if (ctx->use_tc) {     // defined, non-trivial operand planes (see fill_planes_kernel)
        __nv_bfloat16* planes = which == 1 ? kptr<__nv_bfloat16>(ctx, ctx->kl.xa_hl) : which == 3 ? kptr<__nv_bfloat16>(ctx, ctx->kl.act_hl)
                                           : kptr<__nv_bfloat16>(ctx, ctx->kl.xn_hl);
        fill_planes_kernel<<<64, 256, 0, ctx->stream>>>(planes, (size_t)2 * ROWS * K);
        ctx->launches++;
    }
    for (int i = 0; i < 3; ++i) ST(run_gemm<T>(ctx, mr_of(n_rows), site(i), &S));
    CU(cudaEventRecord(ctx->ev[0], ctx->stream));
    for (int i = 0; i < iters; ++i) ST(run_gemm<T>(ctx, mr_of(n_rows), site(i + 3), &S));
    CU(cudaEventRecord(ctx->ev[1], ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    float t = 0.f;
    CU(cudaEventElapsedTime(&t, ctx->ev[0], ctx->ev[1]));
    *ms = t / (float)iters;
    *bytes = (double)N * K * sizeof(T);
    DevState hs;
    return read_state(ctx, &hs);
}

extern "C" {

swift_status swift_time_gemm(swift_ctx* ctx, int32_t which, int32_t n_rows, int32_t iters, float* ms, double* bytes)
{
    if (!ctx || !ms || !bytes) return fail(ctx, SWIFT_EINVAL, "null argument");
    if (ctx->round_open) return fail(ctx, SWIFT_ESTATE, "a round is open");
    if (which < 0 || which > 4 || n_rows < 1 || (n_rows > ROWS && (n_rows % TC_ROWS_MAX || n_rows > TC_BIG_ROWS)) || iters < 1) return fail(ctx, SWIFT_EINVAL, "bad which / n_rows / iters");
    if (ctx->d.dtype == SWIFT_BF16) return time_gemm_t<__nv_bfloat16>(ctx, which, n_rows, iters, ms, bytes);
    return time_gemm_t<float>(ctx, which, n_rows, iters, ms, bytes);
}

swift_status swift_generate(swift_ctx* ctx, const swift_gen_params* gp, const int32_t* prompt, int32_t n_prompt,
                            int32_t* out_tokens, int32_t* n_out, int32_t* trace, swift_stats* stats)
{
    if (!ctx) return SWIFT_EINVAL;
    if (!gp || !prompt || !out_tokens) return fail(ctx, SWIFT_EINVAL, "null argument");
    const swift_model_desc& d = ctx->d;
    if (gp->max_new < 1) return fail(ctx, SWIFT_EINVAL, "max_new must be >= 1");
    if (n_prompt + gp->max_new + 1 > d.max_positions) return fail(ctx, SWIFT_ECAPACITY, "prompt + max_new exceeds max_positions");
    if (!gp->vanilla && tree_active(ctx) && n_prompt + gp->max_new + ctx->tree_rows > d.max_positions)
        return fail(ctx, SWIFT_ECAPACITY, "prompt + max_new + tree_rows exceeds max_positions (the rows of a token tree occupy cache slots)");
    if (!gp->vanilla) {
        if (!gp->skip_mask) return fail(ctx, SWIFT_EINVAL, "skip_mask is null");
        if (gp->max_draft < 0 || gp->max_draft > d.max_draft) return fail(ctx, SWIFT_ECAPACITY, "max_draft %d outside 0..%d", gp->max_draft, d.max_draft);
        if (gp->n_opt_rounds > 0) {
            if (gp->n_candidates < 1 || gp->n_candidates > 1023) return fail(ctx, SWIFT_EINVAL, "n_candidates must be in 1..1023");
            if (!gp->candidate_masks && (gp->opt_skip_blocks < 1 || gp->opt_skip_blocks >= d.n_blocks || gp->opt_beta < 0))
                return fail(ctx, SWIFT_EINVAL, "without candidate masks, opt_skip_blocks must be in 1..n_blocks-1 and opt_beta >= 0");
            if (gp->gamma < 1 || gp->gamma > MAX_SCORE_ROWS) return fail(ctx, SWIFT_ECAPACITY, "gamma must be in 1..%d", MAX_SCORE_ROWS);
        }
    }
    const int L = 2 * d.n_blocks;
    const int64_t launches0 = ctx->launches, h2d0 = ctx->h2d_bytes, d2h0 = ctx->d2h_bytes;
    swift_stats stt;
    memset(&stt, 0, sizeof stt);
    stt.best_matchness = -1.f;
    cudaEvent_t* ev = ctx->ev;
    ctx->round_times.clear();

    CU(cudaEventRecord(ev[0], ctx->stream));
    int first = 0;
    ST(swift_prefill(ctx, prompt, n_prompt, &first));
    CU(cudaEventRecord(ev[1], ctx->stream));
    int count = 0;
    out_tokens[count++] = first;

    std::vector<uint8_t> z(L, 0);
    if (!gp->vanilla) memcpy(z.data(), gp->skip_mask, L);
    bool optimising = !gp->vanilla && gp->n_opt_rounds > 0;
    std::vector<int> counts;
    std::vector<uint8_t> round_masks;
    int stale_rounds = 0;
    // proposals come from the caller, or from the library's own engine (random search + Gaussian-process step)
    // The engine and everything it has learnt stay with the context from one call to the next (the paper optimises over a
    // stream of inputs, Section 4.1's timeline); other settings (blocks to skip, beta, seed) start a new one.
    const bool own_proposals = !gp->vanilla && gp->n_opt_rounds > 0 && !gp->candidate_masks;
    if (own_proposals) {
        const int m_skip = std::max(1, std::min(d.n_blocks - 1, gp->opt_skip_blocks));
        if (!ctx->engine || ctx->engine->m != m_skip || ctx->engine->beta != gp->opt_beta || ctx->engine->seed != gp->opt_seed) {
            delete ctx->engine;
            ctx->engine = new swopt::LayerOpt(d.n_blocks, m_skip, gp->opt_beta, gp->opt_seed);
        }
    }
    swopt::LayerOpt* engine_p = ctx->engine;
    DevState hs;
    while (count < gp->max_new) {
        const int remaining = gp->max_new - count;
        const int n_start = ctx->n;
        if (gp->vanilla) {
            ctx->round++;
            launch_begin_round(ctx, 0.f);
            CU(cudaEventRecord(ev[5], ctx->stream));
            ST(enqueue_verify(ctx, 1, 0));
            if (ctx->mode == SWIFT_SAMPLING) {
                sample_row_kernel<<<1, VOCAB_THREADS, 0, ctx->stream>>>(state_of(ctx), kptr<float>(ctx, ctx->kl.logits), d.vocab, 0,
                                                                        1.0f / ctx->temperature, ctx->seed, (uint32_t)ctx->round, 0u);
                ctx->launches++;
            } else {
                const int save = ctx->mode;
                ST(enqueue_accept(ctx));
                ctx->mode = save;
            }
            CU(cudaEventRecord(ev[6], ctx->stream));
            ST(read_state(ctx, &hs));
            hs.n_accepted = 0;
            float mv = 0.f;
            CU(cudaEventElapsedTime(&mv, ev[5], ev[6]));
            const double bv = forward_bytes(ctx, nullptr, 1, n_start);
            stt.ms_verify += mv;
            stt.bytes_verify += bv;
            ctx->round_times.push_back({0.f, mv, 0.0, bv, 0, 0.0, forward_bytes(ctx, nullptr, 1, n_start, 0)});
        } else {
            if (optimising && count >= gp->gamma) {
                CU(cudaEventRecord(ev[2], ctx->stream));
                // entry 0 is the set in use, scored on the same window as the round's proposals
                const int n_scored = gp->n_candidates + 1;
                round_masks.resize((size_t)n_scored * L);
                memcpy(round_masks.data(), z.data(), L);
                if (own_proposals)
                    for (int c = 0; c < gp->n_candidates; ++c) blocks_to_mask(engine_p->suggest(), d.n_blocks, round_masks.data() + (size_t)(c + 1) * L);
                else
                    memcpy(round_masks.data() + L, gp->candidate_masks + (size_t)stt.opt_rounds * gp->n_candidates * L, (size_t)gp->n_candidates * L);
                const uint8_t* masks = round_masks.data();
                ST(enqueue_score(ctx, masks, n_scored, gp->gamma));
                counts.resize(n_scored);
                CU(copy_async(ctx, counts.data(), kptr<int>(ctx, ctx->kl.score_out), n_scored * 4, cudaMemcpyDeviceToHost));
                CU(cudaEventRecord(ev[3], ctx->stream));
                CU(cudaStreamSynchronize(ctx->stream));
                float ms = 0.f;
                CU(cudaEventElapsedTime(&ms, ev[2], ev[3]));
                stt.ms_score += ms;
                if (own_proposals)                  // every score of the round goes into the Gaussian-process model
                    for (int c = 0; c < n_scored; ++c)
                        engine_p->observe(mask_to_blocks(masks + (size_t)c * L, d.n_blocks), (double)counts[c] / (double)gp->gamma);
                int cb = 0;
                for (int c = 1; c < n_scored; ++c) if (counts[c] > counts[cb]) cb = c;   // strictly better only: the set in use wins ties
                stt.best_matchness = (float)counts[cb] / (float)gp->gamma;
                if (cb != 0) memcpy(z.data(), masks + (size_t)cb * L, L);
                stale_rounds = cb != 0 ? 0 : stale_rounds + 1;
                stt.opt_rounds++;
                if (stt.best_matchness > gp->stop_matchness || stt.opt_rounds >= gp->n_opt_rounds ||
                    (gp->opt_patience > 0 && stale_rounds >= gp->opt_patience))
                    optimising = false;
            }
            const int k_max = std::min(gp->max_draft, remaining - 1);
            CU(cudaEventRecord(ev[4], ctx->stream));
            ST(enqueue_draft(ctx, z.data(), k_max, gp->stop_conf));
            CU(cudaEventRecord(ev[5], ctx->stream));
            ST(enqueue_verify(ctx, k_max + 1, -1));
            ST(enqueue_accept(ctx));
            CU(cudaEventRecord(ev[6], ctx->stream));
            ST(read_state(ctx, &hs));
            float md = 0.f, mv = 0.f;
            CU(cudaEventElapsedTime(&md, ev[4], ev[5]));
            CU(cudaEventElapsedTime(&mv, ev[5], ev[6]));
            stt.ms_draft += md; stt.ms_verify += mv;
            double bd = 0.0;
            for (int j = 0; j < hs.n_drafted; ++j) bd += forward_bytes(ctx, z.data(), 1, n_start + j);
            const int v_rows = hs.tree_rows > 0 ? hs.tree_rows : hs.n_drafted + 1;
            const double bv = forward_bytes(ctx, nullptr, v_rows, n_start);
            stt.bytes_draft += bd;
            stt.bytes_verify += bv;
            double sd = 0.0;                      // the same forwards with the cache counted as it is stored
            for (int j = 0; j < hs.n_drafted; ++j) sd += forward_bytes(ctx, z.data(), 1, n_start + j, 0);
            ctx->round_times.push_back({md, mv, bd, bv, hs.n_drafted, sd, forward_bytes(ctx, nullptr, v_rows, n_start, 0)});
            stt.drafted += hs.n_drafted;
            stt.accepted += hs.n_accepted;
        }
        if (trace) {
            trace[4 * stt.rounds + 0] = n_start; trace[4 * stt.rounds + 1] = gp->vanilla ? 0 : hs.n_drafted;
            trace[4 * stt.rounds + 2] = hs.n_accepted; trace[4 * stt.rounds + 3] = hs.next_token;
        }
        stt.rounds++;
        for (int j = 1; j <= hs.n_accepted; ++j) out_tokens[count++] = hs.draft_tok[j];
        out_tokens[count++] = hs.next_token;
        commit_round(ctx, hs);
    }
    ctx->last_mask = z;
    CU(cudaEventRecord(ev[7], ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    CU(cudaEventElapsedTime(&stt.ms_prefill, ev[0], ev[1]));
    CU(cudaEventElapsedTime(&stt.ms_decode, ev[1], ev[7]));
    stt.tokens = count;
    stt.kernel_launches = ctx->launches - launches0;
    stt.h2d_bytes = ctx->h2d_bytes - h2d0 + (int64_t)n_prompt * 4;     // the prompt itself is read from host memory
    stt.d2h_bytes = ctx->d2h_bytes - d2h0 + (int64_t)count * 4;        // and the tokens are written there
    if (n_out) *n_out = count;
    if (stats) *stats = stt;
    return SWIFT_OK;
}

} // extern "C"
