// Vocabulary-wide kernels: logits reduction + argmax + softmax statistics (+ draft sampling), the
// acceptance step (greedy prefix match or speculative sampling), and the matchness count.
#pragma once
#include "common.cuh"

namespace swk {

constexpr int VOCAB_THREADS = 1024;

struct ArgMax { float v; int i; };
__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b)   // larger value; lowest index on ties
{
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

// Block-wide inverse-CDF draw in index order: smallest i with sum_{i' <= i} w(i') > u * total.
// Thread t owns the contiguous index range [t*seg, (t+1)*seg); its bracket on the running-sum axis
// is [incl(t-1), incl(t)) with both ends read from the same shared array, so the brackets tile
// [0, total) without gaps whatever the rounding.  `sh` is shared scratch of VOCAB_THREADS + 72
// floats.  Every thread returns the same index.  Must be called by all threads of the block.
template <typename WeightFn>
__device__ int block_categorical(WeightFn w, int n, float u, float* sh)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int seg = (n + VOCAB_THREADS - 1) / VOCAB_THREADS;
    const int b = min(tid * seg, n), e = min(b + seg, n);
    float* sh_incl = sh;                                        // [VOCAB_THREADS]
    float* sh_wtot = sh + VOCAB_THREADS;                        // [32]
    int* result = reinterpret_cast<int*>(sh + VOCAB_THREADS + 64);
    float local = 0.f;
    for (int i = b; i < e; ++i) local += w(i);
    float incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                                            // scratch may still be in use by the caller
    if (lane == 31) sh_wtot[warp] = incl;
    if (tid == 0) *result = 0x7FFFFFFF;
    __syncthreads();
    float warp_off = 0.f;
    for (int ww = 0; ww < warp; ++ww) warp_off += sh_wtot[ww];  // sequential, identical for a whole warp
    incl += warp_off;
    sh_incl[tid] = incl;
    __syncthreads();
    const float excl = tid > 0 ? sh_incl[tid - 1] : 0.f;
    const float total = sh_incl[VOCAB_THREADS - 1];
    const float target = u * total;
    if (excl <= target && target < incl) {
        float c = excl;
        int pick = -1, last_pos = -1;
        for (int i = b; i < e; ++i) {
            const float wi = w(i);
            if (wi > 0.f) last_pos = i;
            c += wi;
            if (c > target) { pick = i; break; }
        }
        if (pick < 0) pick = last_pos;                          // rounding at the segment's end
        if (pick >= 0) atomicMin(result, pick);
    }
    __syncthreads();
    if (*result == 0x7FFFFFFF) {
        // nothing bracketed the target (u * total rounded up to the total, or an all-zero row):
        // take the last index that carries weight
        int last = -1;
        for (int i = b; i < e; ++i) if (w(i) > 0.f) last = i;
        int* result2 = result + 1;
        if (tid == 0) *result2 = -1;
        __syncthreads();
        if (last >= 0) atomicMax(result2, last);
        __syncthreads();
        const int out2 = *result2;
        __syncthreads();
        return out2 < 0 ? 0 : out2;
    }
    const int out = *result;
    __syncthreads();
    return out;
}

// One CTA per row.  logits[r][i] = sum_s part[s][r][i]; argmax (lowest id on ties), row max,
// sum exp((l-max)/T); confidence p = max softmax at T = 1.
// VOCAB_DRAFT (one row, draft step j): y'_j = argmax, or (sampling == 1) a draw from q_j = softmax(l/T),
// nucleus-cut, whose probabilities are kept in q_rows[j-1][:], or (sampling == 2) the argmax with the point
// mass on it as q_j; records the token and its confidence, and disarms drafting when the confidence is
// below stop_conf.
__global__ void __launch_bounds__(VOCAB_THREADS)
vocab_kernel(DevState* st, const float* __restrict__ part, int n_split, size_t split_stride,
             float* __restrict__ logits, int vocab, float inv_temp, int mode, int sampling, float* __restrict__ q_rows,
             float top_p, int w_cached, int* __restrict__ cand, int* __restrict__ cand_n)
{
    pdl_enter();
    __shared__ float sh[VOCAB_THREADS + 72];
    __shared__ ArgMax sh_am[32];
    const int r = blockIdx.x;
    if (r >= st->n_rows) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* lrow = logits + (size_t)r * vocab;

    // Vocabularies of up to VOCAB_THREADS * VPT entries with a single slab (the tensor-core path) stay in
    // registers: all of a thread's loads are in flight together and nothing is read back from memory for the
    // second pass.  Same per-thread order of operations as the general loops.
    constexpr int VPT = 32;
    const bool in_regs = n_split == 1 && vocab <= VOCAB_THREADS * VPT;
    float vr[VPT];
    ArgMax am{-INFINITY, 0x7FFFFFFF};
    if (in_regs) {
        const float* prow = part + (size_t)r * vocab;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = tid + k * VOCAB_THREADS;
            vr[k] = i < vocab ? __ldcg(prow + i) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = tid + k * VOCAB_THREADS;
            if (i < vocab) {
                const float v = 0.f + vr[k];
                vr[k] = v;
                lrow[i] = v;
                am = better(am, ArgMax{v, i});
            }
        }
    } else {
        for (int i = tid; i < vocab; i += VOCAB_THREADS) {
            float v = 0.f;
            for (int s = 0; s < n_split; ++s) v += part[s * split_stride + (size_t)r * vocab + i];
            lrow[i] = v;
            am = better(am, ArgMax{v, i});
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ArgMax t{__shfl_xor_sync(0xFFFFFFFFu, am.v, o), __shfl_xor_sync(0xFFFFFFFFu, am.i, o)};
        am = better(am, t);
    }
    if (lane == 0) sh_am[warp] = am;
    __syncthreads();
    if (warp == 0) {
        ArgMax t = sh_am[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ArgMax t2{__shfl_xor_sync(0xFFFFFFFFu, t.v, o), __shfl_xor_sync(0xFFFFFFFFu, t.i, o)};
            t = better(t, t2);
        }
        if (lane == 0) sh_am[0] = t;
    }
    __syncthreads();
    am = sh_am[0];
    __syncthreads();

    float s1 = 0.f, sT = 0.f;
    if (in_regs) {
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            if (tid + k * VOCAB_THREADS < vocab) {
                const float dlt = vr[k] - am.v;
                s1 += expf(dlt);
                sT += expf(dlt * inv_temp);
            }
        }
    } else {
        for (int i = tid; i < vocab; i += VOCAB_THREADS) {
            const float dlt = lrow[i] - am.v;
            s1 += expf(dlt);
            sT += expf(dlt * inv_temp);
        }
    }
    s1 = block_sum(s1, sh);
    sT = block_sum(sT, sh);
    const float conf = 1.f / s1;

    // Nucleus sampling (top_p < 1): keep the most probable tokens whose mass first reaches top_p of the whole, all
    // tokens as probable as the last one included.  With w_i = exp((l_i - max) / T) that is {w_i >= theta} for the
    // largest theta whose kept mass is still >= top_p * sum(w).  Positive floats order like their bit patterns, so
    // theta is found by bisection on the bit pattern (31 block-wide sums); the kept mass replaces the row sum.
    float theta = 0.f;
    if (sampling && top_p < 1.f) {
        const float goal = top_p * sT;
        // w_cached: the launch provides vocab floats of dynamic shared memory, and every thread keeps the weights
        // of its own indices there instead of evaluating 31 x vocab exponentials (same values either way)
        extern __shared__ float w_sh[];
        if (w_cached)
            for (int i = tid; i < vocab; i += VOCAB_THREADS) w_sh[i] = expf((lrow[i] - am.v) * inv_temp);
        auto mass_from = [&](unsigned bits) {
            float m = 0.f;                                      // the row as this thread stored it above, same index order
#pragma unroll 1
            for (int i = tid; i < vocab; i += VOCAB_THREADS) {
                const float w = w_cached ? w_sh[i] : expf((lrow[i] - am.v) * inv_temp);
                if (__float_as_uint(w) >= bits) m += w;
            }
            return block_sum(m, sh);
        };
        unsigned lo = 0u, hi = 0x3F800001u;                     // mass_from(lo) >= goal > mass_from(hi) = 0 (w <= 1)
        while (hi - lo > 1u) {
            const unsigned mid = lo + (hi - lo) / 2u;
            if (mass_from(mid) >= goal) lo = mid; else hi = mid;
        }
        theta = __uint_as_float(lo);
        sT = mass_from(lo);
    }
    if (tid == 0) {
        st->argmax[r] = am.i;
        st->row_max[r] = am.v;
        st->row_sum[r] = sT;
        st->row_thresh[r] = theta;
    }
    if (mode != VOCAB_DRAFT || r != 0) return;

    // step index, threshold and random-number coordinates come from the control block, so that one
    // captured launch sequence serves every draft step of every round
    const int draft_j = st->draft_j;
    const float stop_conf = st->stop_conf;
    const uint64_t seed = ((uint64_t)st->seed_hi << 32) | st->seed_lo;
    const uint32_t round = (uint32_t)st->round;
    int y = am.i;
    if (sampling == 2) {
        // greedy drafts under speculative-sampling acceptance (Eq. 4 taken literally): q_j is the point mass on y'_j
        float* qrow = q_rows + (size_t)(draft_j - 1) * vocab;
        for (int i = tid; i < vocab; i += VOCAB_THREADS) qrow[i] = i == y ? 1.f : 0.f;
    } else if (sampling) {
        float* qrow = q_rows + (size_t)(draft_j - 1) * vocab;
        const float inv_sum = 1.f / sT;
        for (int i = tid; i < vocab; i += VOCAB_THREADS) {
            const float w = expf((lrow[i] - am.v) * inv_temp);
            qrow[i] = w >= theta ? w * inv_sum : 0.f;
        }
        __syncthreads();
        const float u = philox_uniform(seed, round, (uint32_t)draft_j, DRAW_DRAFT);
        y = block_categorical([&](int i) { return qrow[i]; }, vocab, u, sh);
    }
    if (tid == 0) {
        st->draft_tok[draft_j] = y;
        st->conf[draft_j - 1] = conf;
        st->n_drafted = draft_j;
        if (conf < stop_conf) st->active = 0;
    }
    // Dynamic verification (Section 4.2): the draft position is extended with the draft model's top-k predictions,
    // k by the confidence of the position.  cand[(j-1)*TREE_TOPK + i] = the i-th best token (logit descending, token
    // id ascending among equals; entry 0 is y'_j itself), found by k - 1 further arg-max passes over the row, each
    // restricted to what ranks after the previous pick.
    if (cand != nullptr && !sampling) {
        const int width = conf <= 0.5f ? 10 : conf <= 0.8f ? 5 : conf <= 0.95f ? 3 : 1;
        if (tid == 0) { cand[(draft_j - 1) * TREE_TOPK] = am.i; cand_n[draft_j - 1] = width; }
        ArgMax prev = am;
        for (int rank = 1; rank < width; ++rank) {
            ArgMax best{-INFINITY, 0x7FFFFFFF};
            for (int i = tid; i < vocab; i += VOCAB_THREADS) {
                const float v = lrow[i];
                if (v < prev.v || (v == prev.v && i > prev.i)) best = better(best, ArgMax{v, i});
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                ArgMax t2{__shfl_xor_sync(0xFFFFFFFFu, best.v, o), __shfl_xor_sync(0xFFFFFFFFu, best.i, o)};
                best = better(best, t2);
            }
            __syncthreads();
            if (lane == 0) sh_am[warp] = best;
            __syncthreads();
            if (warp == 0) {
                ArgMax t3 = sh_am[lane];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    ArgMax t4{__shfl_xor_sync(0xFFFFFFFFu, t3.v, o), __shfl_xor_sync(0xFFFFFFFFu, t3.i, o)};
                    t3 = better(t3, t4);
                }
                if (lane == 0) sh_am[0] = t3;
            }
            __syncthreads();
            prev = sh_am[0];
            if (tid == 0) cand[(draft_j - 1) * TREE_TOPK + rank] = prev.i;
        }
    }
}

// Acceptance over the k = st->n_drafted drafts of the round, one CTA.  `logits` holds the k+1
// target rows, st->argmax / row_max / row_sum their statistics, q_rows the draft distributions.
// Writes n_accepted, next_token, and makes next_token the pending token (draft_tok[0]).
__global__ void __launch_bounds__(VOCAB_THREADS)
accept_kernel(DevState* st, const float* __restrict__ logits, const float* __restrict__ q_rows, int vocab,
              int sampling, float inv_temp, uint64_t seed, uint32_t round)
{
    __shared__ float sh[VOCAB_THREADS + 72];
    __shared__ int sh_a, sh_rejected;
    const int k = st->n_drafted;
    const int tid = threadIdx.x;
    if (!sampling && st->tree_rows > 0) {
        // greedy verification of a token tree: from row 0 follow the child whose token is the target's arg max at the
        // current node; where no child matches, that arg max is the next token
        if (tid == 0) {
            const int rows = st->tree_rows;
            int node = 0, a = 0, gold = st->argmax[0];
            for (;;) {
                gold = st->argmax[node];
                int hit = -1;
                for (int r = 1; r < rows; ++r)
                    if (st->row_parent[r] == node && st->draft_tok[r] == gold) { hit = r; break; }
                if (hit < 0) break;
                st->acc_row[a++] = hit;
                node = hit;
            }
            for (int j = 1; j <= a; ++j) st->draft_tok[j] = st->draft_tok[st->acc_row[j - 1]];   // acc_row[j-1] >= j: read before overwritten
            st->n_accepted = a;
            st->next_token = gold;
            st->draft_tok[0] = gold;
        }
        return;
    }
    if (!sampling) {
        if (tid == 0) {
            int a = 0;
            while (a < k && st->draft_tok[a + 1] == st->argmax[a]) ++a;
            st->n_accepted = a;
            st->next_token = st->argmax[a];
            st->draft_tok[0] = st->argmax[a];
        }
        return;
    }
    if (tid == 0) {
        int a = 0, rejected = 0;
        for (int j = 1; j <= k; ++j) {
            const int y = st->draft_tok[j];
            const float w = expf((logits[(size_t)(j - 1) * vocab + y] - st->row_max[j - 1]) * inv_temp);
            const float p = w >= st->row_thresh[j - 1] ? w / st->row_sum[j - 1] : 0.f;
            const float q = q_rows[(size_t)(j - 1) * vocab + y];
            const float u = philox_uniform(seed, round, (uint32_t)j, DRAW_ACCEPT);
            if (!(u * q < p)) { rejected = 1; break; }
            ++a;
        }
        sh_a = a;
        sh_rejected = rejected;
    }
    __syncthreads();
    const int a = sh_a, rejected = sh_rejected;
    const float* lrow = logits + (size_t)a * vocab;          // target row j-1 with j = a+1
    const float mx = st->row_max[a], inv_sum = 1.f / st->row_sum[a], theta = st->row_thresh[a];
    auto p_of = [&](int i) { const float w = expf((lrow[i] - mx) * inv_temp); return w >= theta ? w * inv_sum : 0.f; };
    int tok;
    if (rejected) {
        const float* qrow = q_rows + (size_t)a * vocab;
        float mass = 0.f;
        for (int i = tid; i < vocab; i += VOCAB_THREADS) mass += fmaxf(p_of(i) - qrow[i], 0.f);
        mass = block_sum(mass, sh);
        const float u = philox_uniform(seed, round, (uint32_t)(a + 1), DRAW_RESAMPLE);
        if (mass > 0.f) tok = block_categorical([&](int i) { return fmaxf(p_of(i) - qrow[i], 0.f); }, vocab, u, sh);
        else tok = block_categorical(p_of, vocab, u, sh);
    } else {
        const float u = philox_uniform(seed, round, (uint32_t)(k + 1), DRAW_BONUS);
        tok = block_categorical(p_of, vocab, u, sh);
    }
    if (tid == 0) {
        st->n_accepted = a;
        st->next_token = tok;
        st->draft_tok[0] = tok;
    }
}

// Draws one token from softmax(row r / T) of the last forward (first token in sampling mode, and
// vanilla sampling steps): counter (round, slot, DRAW_BONUS).
__global__ void __launch_bounds__(VOCAB_THREADS)
sample_row_kernel(DevState* st, const float* __restrict__ logits, int vocab, int row, float inv_temp,
                  uint64_t seed, uint32_t round, uint32_t slot)
{
    __shared__ float sh[VOCAB_THREADS + 72];
    const float* lrow = logits + (size_t)row * vocab;
    const float mx = st->row_max[row], theta = st->row_thresh[row];
    const float u = philox_uniform(seed, round, slot, DRAW_BONUS);
    const int tok = block_categorical([&](int i) { const float w = expf((lrow[i] - mx) * inv_temp); return w >= theta ? w : 0.f; },
                                      vocab, u, sh);
    if (threadIdx.x == 0) {
        st->next_token = tok;
        st->draft_tok[0] = tok;
    }
}

// matchness numerator (Eq. 3): adds #(argmax[r] == truth[r]) over the rows of this chunk; the
// running count is stored to *out after the candidate's last chunk.
__global__ void match_count_kernel(DevState* st, const int* __restrict__ truth, int reset, int* out)
{
    if (threadIdx.x == 0) {
        int c = reset ? 0 : st->match_count;
        for (int r = 0; r < st->n_rows; ++r) c += (st->argmax[r] == truth[r]) ? 1 : 0;
        st->match_count = c;
        if (out) *out = c;
    }
}

} // namespace swk
