// Host-side proposal engine for the on-the-fly layer-set optimisation (Section 4.1, "Efficient Layer Set
// Suggestion"): random search over the sets of m of n_blocks blocks, with a Gaussian-process (Bayesian
// optimisation) proposal every beta-th step.  Plain C++, no device code.
//
// The paper leaves the Bayesian step to a third-party package; this is the textbook form.  A set is its indicator
// vector, the squared distance of two sets their Hamming distance.  Scores are standardised.  Mean function: ridge
// regression of the scores on the indicators over all evaluated sets (what each block costs when skipped).  On the
// residuals of the most recent evaluations: a zero-mean GP with Matern-5/2 covariance
// k(d) = (1 + s + s^2/3) exp(-s), s = sqrt(5) d / ell, plus observation noise; ell is the candidate length scale with the
// highest marginal likelihood; the posterior comes from a Cholesky factorisation.  The proposal is the unevaluated set with
// the highest mean + kappa * deviation among a pool: random sets, all sets one swap away from the best set seen, the m
// blocks with the smallest regression cost and all sets one swap away from that.  Random draws are Philox4x32-10 words.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <set>
#include <thread>
#include <vector>

namespace swopt {

inline void philox_round(uint32_t (&c)[4], uint32_t (&k)[2])
{
    const uint64_t p0 = (uint64_t)0xD2511F53u * c[0], p1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k[0], n1 = (uint32_t)p1, n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k[1], n3 = (uint32_t)p0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
    k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u;
}
// first output word of Philox4x32-10 at counter (index lo, index hi, 7, tag), key = seed
inline uint32_t philox_word(uint64_t seed, uint64_t index)
{
    uint32_t c[4] = {(uint32_t)index, (uint32_t)(index >> 32), 7u, 0x4F5054u};
    uint32_t k[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int r = 0; r < 10; ++r) philox_round(c, k);
    return c[0];
}

typedef std::vector<int> BlockSet;   // sorted block indices

struct GpModel {
    std::vector<BlockSet> X;
    std::vector<double> L, alpha;    // Cholesky factor (row-major lower triangle, n x n) and K^-1 t
    std::vector<double> w;           // mean function: regression weight of every block
    double mu = 0.0, sd = 1.0, ell = 1.0, lml = 0.0;
    int n = 0;
};

class LayerOpt {
public:
    LayerOpt(int n_blocks, int m, int beta, uint64_t seed, int pool = 512, double kappa = 2.576, double noise = 1e-2)
        : nb(n_blocks), m(m), beta(beta), pool(pool), seed(seed), kappa(kappa), noise(noise) {}

    int nb, m, beta, pool;
    uint64_t seed;
    double kappa, noise;
    std::vector<double> ells = {1.0, 2.0, 4.0};
    double ridge = 1.0;              // regularisation of the mean function
    int gp_window = 256;             // the GP sees the residuals of this many most recent evaluations
    long long step = 0;              // proposals made
    uint64_t draws = 0;              // random words consumed
    std::vector<BlockSet> X;         // evaluated sets ...
    std::vector<double> y;           // ... and their matchness

    BlockSet random_set()
    {
        std::vector<int> idx(nb);
        for (int i = 0; i < nb; ++i) idx[i] = i;
        for (int i = 0; i < m; ++i) {               // partial Fisher-Yates shuffle
            const int j = i + (int)(philox_word(seed, draws++) % (uint32_t)(nb - i));
            std::swap(idx[i], idx[j]);
        }
        BlockSet s(idx.begin(), idx.begin() + m);
        std::sort(s.begin(), s.end());
        return s;
    }

    static int hamming(const BlockSet& a, const BlockSet& b)   // of the indicator vectors
    {
        size_t i = 0, j = 0;
        int common = 0;
        while (i < a.size() && j < b.size()) {
            if (a[i] == b[j]) { ++common; ++i; ++j; }
            else if (a[i] < b[j]) ++i;
            else ++j;
        }
        return (int)a.size() + (int)b.size() - 2 * common;
    }
    static double matern52(double d2, double ell)
    {
        const double s = std::sqrt(5.0 * d2) / ell;
        return (1.0 + s + s * s / 3.0) * std::exp(-s);
    }

    int best_index() const                           // highest matchness, the earliest among equals
    {
        int b = -1;
        for (size_t i = 0; i < y.size(); ++i)
            if (b < 0 || y[i] > y[b]) b = (int)i;
        return b;
    }

    void observe(const BlockSet& s, double matchness)
    {
        BlockSet t(s);
        std::sort(t.begin(), t.end());
        X.push_back(t);
        y.push_back(matchness);
    }

    GpModel fit() const;
    void predict(const GpModel& g, const BlockSet& s, double* mean, double* dev) const;
    BlockSet bayesian_set(double* ucb_out = nullptr);
    BlockSet suggest()
    {
        ++step;
        if (beta > 0 && step % beta == 0 && !X.empty()) return bayesian_set();
        return random_set();
    }
};

// fn(i) for i in [0, n) on up to eight host threads (contiguous ranges); the calls must not depend on one another.
template <typename F>
inline void parallel_for(int n, F fn)
{
    const int hw = (int)std::thread::hardware_concurrency();
    const int T = std::max(1, std::min(std::min(8, hw > 0 ? hw : 1), n));
    if (T == 1) {
        for (int i = 0; i < n; ++i) fn(i);
        return;
    }
    std::vector<std::thread> th;
    for (int k = 0; k < T; ++k)
        th.emplace_back([&, k] { for (int i = (int)((long long)n * k / T); i < (int)((long long)n * (k + 1) / T); ++i) fn(i); });
    for (std::thread& x : th) x.join();
}

inline GpModel LayerOpt::fit() const
{
    const int n_all = (int)y.size();
    GpModel best;
    double mu = 0.0, var = 0.0;
    for (double v : y) mu += v;
    mu /= n_all;
    for (double v : y) var += (v - mu) * (v - mu);
    double sd = std::sqrt(var / n_all);
    if (sd <= 1e-12) sd = 1.0;
    std::vector<double> t_all(n_all);
    for (int i = 0; i < n_all; ++i) t_all[i] = (y[i] - mu) / sd;
    // mean function: (X^T X + ridge I) w = X^T t over all evaluations, by Cholesky of the n_blocks x n_blocks matrix
    std::vector<double> A((size_t)nb * nb, 0.0), w(nb, 0.0);
    for (int i = 0; i < n_all; ++i)
        for (int p : X[i]) {
            w[p] += t_all[i];
            for (int q : X[i]) A[(size_t)p * nb + q] += 1.0;
        }
    for (int p = 0; p < nb; ++p) A[(size_t)p * nb + p] += ridge;
    for (int i = 0; i < nb; ++i)
        for (int j = 0; j <= i; ++j) {
            double acc = A[(size_t)i * nb + j];
            for (int k = 0; k < j; ++k) acc -= A[(size_t)i * nb + k] * A[(size_t)j * nb + k];
            A[(size_t)i * nb + j] = i == j ? std::sqrt(acc) : acc / A[(size_t)j * nb + j];
        }
    for (int i = 0; i < nb; ++i) {
        for (int k = 0; k < i; ++k) w[i] -= A[(size_t)i * nb + k] * w[k];
        w[i] /= A[(size_t)i * nb + i];
    }
    for (int i = nb - 1; i >= 0; --i) {
        for (int k = i + 1; k < nb; ++k) w[i] -= A[(size_t)k * nb + i] * w[k];
        w[i] /= A[(size_t)i * nb + i];
    }
    // the GP models the residuals of the most recent evaluations
    const int n = std::min(n_all, gp_window), first = n_all - n;
    std::vector<double> t(n), d2((size_t)n * n);
    for (int i = 0; i < n; ++i) {
        double r = t_all[first + i];
        for (int p : X[first + i]) r -= w[p];
        t[i] = r;
    }
    for (int i = 0; i < n; ++i)
        for (int j = 0; j <= i; ++j) d2[(size_t)i * n + j] = hamming(X[first + i], X[first + j]);
    // one factorisation per length scale, side by side on host threads; the choice among them is made in the scales' order
    struct Trial { std::vector<double> L, a; double lml = 0.0; bool ok = false; };
    std::vector<Trial> trials(ells.size());
    parallel_for((int)ells.size(), [&](int e) {
        const double ell = ells[e];
        Trial& tr = trials[e];
        std::vector<double> Lc((size_t)n * n, 0.0);
        bool ok = true;
        for (int i = 0; i < n && ok; ++i) {           // Cholesky, row by row
            for (int j = 0; j <= i; ++j) {
                double acc = matern52(d2[(size_t)i * n + j], ell) + (i == j ? noise : 0.0);
                for (int k = 0; k < j; ++k) acc -= Lc[(size_t)i * n + k] * Lc[(size_t)j * n + k];
                if (i == j) {
                    if (acc <= 0.0) { ok = false; break; }
                    Lc[(size_t)i * n + i] = std::sqrt(acc);
                } else {
                    Lc[(size_t)i * n + j] = acc / Lc[(size_t)j * n + j];
                }
            }
        }
        if (!ok) return;
        std::vector<double> a(t);                     // alpha = K^-1 t by two triangular solves
        for (int i = 0; i < n; ++i) {
            for (int k = 0; k < i; ++k) a[i] -= Lc[(size_t)i * n + k] * a[k];
            a[i] /= Lc[(size_t)i * n + i];
        }
        for (int i = n - 1; i >= 0; --i) {
            for (int k = i + 1; k < n; ++k) a[i] -= Lc[(size_t)k * n + i] * a[k];
            a[i] /= Lc[(size_t)i * n + i];
        }
        double lml = -0.5 * n * std::log(2.0 * 3.14159265358979323846);
        for (int i = 0; i < n; ++i) lml -= 0.5 * t[i] * a[i] + std::log(Lc[(size_t)i * n + i]);
        tr.L.swap(Lc); tr.a.swap(a); tr.lml = lml; tr.ok = true;
    });
    bool have = false;
    for (size_t e = 0; e < ells.size(); ++e) {
        Trial& tr = trials[e];
        if (tr.ok && (!have || tr.lml > best.lml)) {
            have = true;
            best.L.swap(tr.L); best.alpha.swap(tr.a); best.ell = ells[e]; best.lml = tr.lml;
        }
    }
    best.X.assign(X.begin() + first, X.end());
    best.w = w; best.mu = mu; best.sd = sd; best.n = have ? n : 0;
    return best;
}

inline void LayerOpt::predict(const GpModel& g, const BlockSet& s, double* mean, double* dev) const
{
    const int n = g.n;
    std::vector<double> ks(n), v(n);
    double mu = 0.0;
    for (int i = 0; i < n; ++i) { ks[i] = matern52(hamming(s, g.X[i]), g.ell); mu += ks[i] * g.alpha[i]; }
    double q = 0.0;                                   // |L^-1 ks|^2
    for (int i = 0; i < n; ++i) {
        double acc = ks[i];
        for (int k = 0; k < i; ++k) acc -= g.L[(size_t)i * n + k] * v[k];
        v[i] = acc / g.L[(size_t)i * n + i];
        q += v[i] * v[i];
    }
    for (int p : s) mu += g.w[p];                     // mean function
    *mean = g.mu + g.sd * mu;
    *dev = g.sd * std::sqrt(std::max(1.0 - q, 0.0));
}

inline BlockSet LayerOpt::bayesian_set(double* ucb_out)
{
    std::vector<BlockSet> cand;
    for (int i = 0; i < pool; ++i) cand.push_back(random_set());
    auto add_swaps = [&](const BlockSet& base) {      // every set one swap away from `base`
        std::vector<int> outside;
        for (int b = 0; b < nb; ++b) if (!std::binary_search(base.begin(), base.end(), b)) outside.push_back(b);
        for (int out_b : base)
            for (int in_b : outside) {
                BlockSet s;
                for (int b : base) if (b != out_b) s.push_back(b);
                s.push_back(in_b);
                std::sort(s.begin(), s.end());
                cand.push_back(s);
            }
    };
    const int bi = best_index();
    GpModel g;
    if (!X.empty()) g = fit();
    if (bi >= 0) {
        add_swaps(X[bi]);
        // the m blocks that cost least to skip according to the regression: largest weights, compared to six decimals
        // (blocks that were always skipped together get the same weight up to rounding), lowest index among equals
        std::vector<int> order(nb);
        std::vector<long long> key(nb);
        for (int b = 0; b < nb; ++b) { order[b] = b; key[b] = (long long)std::floor(g.w[b] * 1e6 + 0.5); }
        std::stable_sort(order.begin(), order.end(), [&](int p, int q) { return key[p] > key[q]; });
        BlockSet cheapest(order.begin(), order.begin() + m);
        std::sort(cheapest.begin(), cheapest.end());
        cand.push_back(cheapest);
        add_swaps(cheapest);
    }
    std::set<BlockSet> seen(X.begin(), X.end());      // leave out evaluated sets and repeats, keeping pool order
    std::vector<BlockSet> fresh;
    for (const BlockSet& c : cand)
        if (seen.insert(c).second) fresh.push_back(c);
    if (fresh.empty()) return random_set();
    if (X.empty() || g.n == 0) return fresh[0];
    std::vector<double> ucb(fresh.size());             // each prediction is independent: host threads, same values as in turn
    parallel_for((int)fresh.size(), [&](int i) {
        double mean, dev;
        predict(g, fresh[i], &mean, &dev);
        ucb[i] = mean + kappa * dev;
    });
    int pick = 0;
    double best = 0.0;
    for (size_t i = 0; i < fresh.size(); ++i)
        if (i == 0 || ucb[i] > best) { best = ucb[i]; pick = (int)i; }
    if (ucb_out) *ucb_out = best;
    return fresh[pick];
}

} // namespace swopt
