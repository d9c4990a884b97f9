// Host side of the code model: format arithmetic and the table of integer symbol weights of the
// quantised generalized-normal source (Sec. III (ii): the Huffman code is designed from the
// GenNorm model of the converted gradient; Sec. IV-B "Huffman coding").
//
// The table T[ibeta][ir][j] is a pure function of the format.  For shape beta_q = 2^(ibeta/8)
// and scale (relative to the bias) r_q = ir/8, the cell of magnitude code j is bounded by the
// midpoints to its neighbours; its probability is a difference of the GenNorm CDF
// Pr(|X| <= t) = P(1/beta, (t/alpha)^beta) (regularised lower incomplete gamma).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "co3_internal.h"

int co3_host_fmt_ok(co3_format f) {
    return f.exp_bits >= 1 && f.exp_bits <= 4 && f.mant_bits >= 1 && f.exp_bits + f.mant_bits <= 7;
}

int co3_host_cF(int E, int M) { return 1 - ((1 << (E - 1)) - 1) - M; }

int64_t co3_host_K(int M, int j) {
    int e = j >> M, f = j & ((1 << M) - 1);
    return e == 0 ? (int64_t)f : ((int64_t)((1 << M) + f) << (e - 1));
}

namespace {

// lower series: gamma(a,x) = x^a e^-x sum_{n>=0} x^n / (a (a+1) ... (a+n))
double lower_series(double a, double x, double log_pref) {
    double denom = a, term = 1.0 / a, total = term;
    for (int n = 1; n < 200000; ++n) {
        denom += 1.0;
        term = term * x / denom;
        total += term;
        if (term <= total * 5e-18) break;
    }
    return total * exp(log_pref);
}

// upper continued fraction, evaluated with the forward (Wallis) recurrence and rescaling:
// Gamma(a,x) = x^a e^-x * 1/(x+1-a - 1(1-a)/(x+3-a - 2(2-a)/(x+5-a - ...)))
double upper_fraction(double a, double x, double log_pref) {
    // Write the fraction as 1/f, f = b0 + a1/(b1 + a2/(b2 + ...)); convergents A_i/B_i of f with
    // A_{-1} = 1, A_0 = b0, B_{-1} = 0, B_0 = 1.
    const double b0 = x + 1.0 - a;
    double Am1 = 1.0, A0 = b0, Bm1 = 0.0, B0 = 1.0;
    double prev = A0 / B0;
    for (int i = 1; i < 200000; ++i) {
        double ai = -(double)i * ((double)i - a);
        double bi = x + (double)(2 * i + 1) - a;
        double A1 = bi * A0 + ai * Am1;
        double B1 = bi * B0 + ai * Bm1;
        Am1 = A0; A0 = A1; Bm1 = B0; B0 = B1;
        if (fabs(A0) > 1e200 || fabs(B0) > 1e200) {
            Am1 *= 1e-200; A0 *= 1e-200; Bm1 *= 1e-200; B0 *= 1e-200;
        }
        if (B0 != 0.0) {
            double cur = A0 / B0;
            if (fabs(cur - prev) <= fabs(cur) * 1e-16) { prev = cur; break; }
            prev = cur;
        }
    }
    return exp(log_pref) / prev;
}

double reg_lower_gamma(double a, double x) {
    if (!(x > 0.0)) return 0.0;
    if (isinf(x)) return 1.0;
    double log_pref = a * log(x) - x - lgamma(a);
    if (x < a + 1.0) {
        double p = lower_series(a, x, log_pref);
        return p > 1.0 ? 1.0 : p;
    }
    double q = upper_fraction(a, x, log_pref);
    if (q < 0.0) q = 0.0;
    if (q > 1.0) q = 1.0;
    return 1.0 - q;
}

void weight_row(int E, int M, int ibeta, int ir, uint32_t* half /* J entries */) {
    const int J = 1 << (E + M);
    const double beta_q = exp2((double)ibeta / 8.0), r_q = (double)ir / 8.0;
    const double unit = exp2((double)co3_host_cF(E, M) - r_q);
    const double scale = 1048576.0;
    double below = 0.0;
    for (int j = 0; j < J; ++j) {
        double cdf = 1.0;
        if (j < J - 1) {
            double tau = 0.5 * (double)(co3_host_K(M, j) + co3_host_K(M, j + 1)) * unit;
            cdf = reg_lower_gamma(1.0 / beta_q, pow(tau, beta_q));
        }
        double mass = cdf - below;
        below = cdf;
        double x = (j == 0) ? floor(scale * mass + 0.5) : floor(scale * mass / 2.0 + 0.5);
        half[j] = x < 1.0 ? 1u : (uint32_t)x;
    }
}

// Expected squared conversion error of X ~ GenNorm(alpha, beta_q), divided by alpha^2, when
// log2(alpha) - b = ir/8 (the L2 objective of Eq. "exp bias" on the header grid).  Computed edge by
// edge: at every cell edge t (in units of alpha) the three partial moments
//   m_k(t) = int_0^t x^k dF = Gamma((k+1)/beta)/Gamma(1/beta) * P((k+1)/beta, t^beta),  k = 0, 1, 2
// are evaluated once, and the cell between two edges adds (dm2 - 2 v dm1 + v^2 dm0) for its grid
// value v; beyond the last edge (saturation) the moments are their totals.
double grid_distortion(int E, int M, int ibeta, int ir) {
    const int J = 1 << (E + M);
    const double beta_q = exp2((double)ibeta / 8.0);
    const double unit = exp2((double)co3_host_cF(E, M) - (double)ir / 8.0);   // grid quantum / alpha
    const double s0 = 1.0 / beta_q, s1 = 2.0 / beta_q, s2 = 3.0 / beta_q;
    const double g1 = exp(lgamma(s1) - lgamma(s0)), g2 = exp(lgamma(s2) - lgamma(s0));
    double lo[3] = {0.0, 0.0, 0.0}, sum = 0.0;
    for (int j = 0; j < J; ++j) {
        double hi[3] = {1.0, g1, g2};
        if (j + 1 < J) {
            const double edge = 0.5 * (double)(co3_host_K(M, j) + co3_host_K(M, j + 1)) * unit;
            const double z = pow(edge, beta_q);
            hi[0] = reg_lower_gamma(s0, z);
            hi[1] = g1 * reg_lower_gamma(s1, z);
            hi[2] = g2 * reg_lower_gamma(s2, z);
        }
        const double v = (double)co3_host_K(M, j) * unit;
        sum += (hi[2] - lo[2]) - 2.0 * v * (hi[1] - lo[1]) + v * v * (hi[0] - lo[0]);
        lo[0] = hi[0]; lo[1] = hi[1]; lo[2] = hi[2];
    }
    return sum;
}

struct TableCache {
    int E, M;
    uint32_t* data;
};
struct OptCache {
    int E, M;
    int16_t tab[CO3_NIBETA * 8];
};
OptCache g_opt[16];
int g_nopt = 0;
TableCache g_cache[16];
int g_ncache = 0;
std::mutex g_mu;

}  // namespace

const uint32_t* co3_host_weight_table(int E, int M) {
    std::lock_guard<std::mutex> lk(g_mu);
    for (int i = 0; i < g_ncache; ++i)
        if (g_cache[i].E == E && g_cache[i].M == M) return g_cache[i].data;
    if (g_ncache == 16) return nullptr;
    const int J = 1 << (E + M);
    uint32_t* t = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)CO3_NIBETA * CO3_NIR * J);
    if (!t) return nullptr;
    for (int ib = 0; ib < CO3_NIBETA; ++ib)
        for (int r = 0; r < CO3_NIR; ++r)
            weight_row(E, M, ib + CO3_IBETA_MIN, r + CO3_IR_MIN, t + ((size_t)ib * CO3_NIR + r) * J);
    g_cache[g_ncache++] = TableCache{E, M, t};
    return t;
}

// Bias rule "optimal": moving b by one moves ir by eight, so the L2-best integer bias for a shape
// index and a residue rho = round(8 log2 alpha) mod 8 is the ir of least distortion among those
// congruent to rho (the first one in ascending ir on an exact tie).  [NIBETA][8] entries, cached.
const int16_t* co3_host_bias_opt_table(int E, int M) {
    std::lock_guard<std::mutex> lk(g_mu);
    for (int i = 0; i < g_nopt; ++i)
        if (g_opt[i].E == E && g_opt[i].M == M) return g_opt[i].tab;
    if (g_nopt == 16) return nullptr;
    OptCache& c = g_opt[g_nopt];
    c.E = E; c.M = M;
    for (int ib = 0; ib < CO3_NIBETA; ++ib) {
        double best[8];
        int arg[8];
        for (int k = 0; k < 8; ++k) { best[k] = -1.0; arg[k] = 0; }
        for (int ir = CO3_IR_MIN; ir <= CO3_IR_MAX; ++ir) {
            const int rho = ((ir % 8) + 8) % 8;
            const double dist = grid_distortion(E, M, ib + CO3_IBETA_MIN, ir);
            if (best[rho] < 0.0 || dist < best[rho]) { best[rho] = dist; arg[rho] = ir; }
        }
        for (int k = 0; k < 8; ++k) c.tab[ib * 8 + k] = (int16_t)arg[k];
    }
    ++g_nopt;
    return c.tab;
}

extern "C" int co3_bias_opt_table(co3_format fmt, int16_t* table) {
    if (!co3_host_fmt_ok(fmt) || !table) return CO3_EINVAL;
    const int16_t* t = co3_host_bias_opt_table(fmt.exp_bits, fmt.mant_bits);
    if (!t) return CO3_ENOMEM;
    memcpy(table, t, sizeof(int16_t) * CO3_NIBETA * 8);
    return CO3_OK;
}

extern "C" double co3_grid_distortion(co3_format fmt, int32_t ibeta, int32_t ir) {
    if (!co3_host_fmt_ok(fmt) || ibeta < CO3_IBETA_MIN || ibeta > CO3_IBETA_MAX || ir < CO3_IR_MIN || ir > CO3_IR_MAX)
        return -1.0;
    return grid_distortion(fmt.exp_bits, fmt.mant_bits, ibeta, ir);
}

// Two functions of the GenNorm shape on a grid uniform in log2(beta) over [log2 0.3, log2 2]:
//   [0 .. FIT_GRID]              log R(beta) = lgamma(1/b) + lgamma(3/b) - 2 lgamma(2/b)
//   [FIT_GRID+1 .. 2 FIT_GRID+1] log G(beta) = lgamma(1/b) - lgamma(2/b)
// The moment ratio of a GenNorm sample is R(beta) (the device inverts the first table by inverse
// cubic interpolation) and its scale is alpha = E|X| * G(beta) (second table, cubic interpolation).
const double* co3_host_logr_table(void) {
    static double* tab = nullptr;
    std::lock_guard<std::mutex> lk(g_mu);
    if (tab) return tab;
    double* t = (double*)malloc(sizeof(double) * 2 * (CO3_FIT_GRID + 1));
    if (!t) return nullptr;
    const double t0 = log2(0.3), t1 = 1.0;
    for (int i = 0; i <= CO3_FIT_GRID; ++i) {
        double b = (i == 0) ? 0.3 : (i == CO3_FIT_GRID ? 2.0 : exp2(t0 + (t1 - t0) * ((double)i / CO3_FIT_GRID)));
        t[i] = lgamma(1.0 / b) + lgamma(3.0 / b) - 2.0 * lgamma(2.0 / b);
        t[CO3_FIT_GRID + 1 + i] = lgamma(1.0 / b) - lgamma(2.0 / b);
    }
    tab = t;
    return tab;
}

extern "C" int co3_model_weights(co3_format fmt, int32_t ibeta, int32_t ir, uint32_t* weights) {
    if (!co3_host_fmt_ok(fmt) || !weights || ibeta < CO3_IBETA_MIN || ibeta > CO3_IBETA_MAX ||
        ir < CO3_IR_MIN || ir > CO3_IR_MAX)
        return CO3_EINVAL;
    const int E = fmt.exp_bits, M = fmt.mant_bits, J = 1 << (E + M);
    uint32_t half[128];
    weight_row(E, M, ibeta, ir, half);
    for (int j = 0; j < J; ++j) {
        weights[j] = half[j];
        weights[J + j] = (j == 0) ? 1u : half[j];   // "-0" is never emitted
    }
    return CO3_OK;
}

// Contiguous split of n work items over at most max_blocks thread blocks for kernels whose blocks walk
// their items run by run of one segment, the block's `teams` teams taking every teams-th item of a run
// and all of them meeting where the segment changes.  A run lasts at least as long as its most loaded
// team needs, and a block whose teams are all busy is bound by the throughput of its SM, i.e. by its
// total work; the time of a run is modelled as the mean of the two (its most loaded team's items, and
// its total / teams) plus run_cost / 2 for the change of tables, and a block takes the sum over its
// runs.  (Per-block cycle counts taken with clock64 on the 62-layer ResNet-18 workload, 8 users, 4
// teams: 20 full chunks in one run 166 k, 19 in one run 145-160 k, 10 + 1 + 2 + 5 chunks in four runs
// of which two are tiny layers 170 k.  A model that takes the larger of 0.45 x the team's items and the
// total / teams fits those counts a little better and gave a kernel 2 % slower on that workload, 3 %
// faster with four users: within what the choice of cuts can move.)  Equal item counts per block let a
// block with a few tiny layers in its range, or one that a layer boundary cuts into 10 + 9, take a
// round more than its neighbours, and every block waits for the slowest; the cuts are therefore placed
// so that the largest block cost is as small as a contiguous split allows (bisection on that bound),
// and within that bound the work is spread over all the blocks in proportion.  part[0 .. max_blocks]
// receives the cuts; returns the blocks in use.
int co3_host_balanced_split(const double* w, const int32_t* seg, int64_t n, int teams, int max_blocks, double run_cost,
                            int32_t* part) {
    if (!w || !seg || !part || n < 1 || n > 0x7FFFFFFFLL || teams < 1 || teams > 32 || max_blocks < 1) return -1;
    auto run_time = [&](double team_max, double work) {
        return 0.5 * team_max + 0.5 * work / teams + 0.5 * run_cost;
    };
    // furthest end (exclusive) of a block that starts at item `from` and costs at most `bound`
    auto reach = [&](int64_t from, double bound) {
        int64_t i = from;
        double closed = 0.0, team_sum[32] = {0}, run_max = w[i], run_work = w[i];   // a block takes at least one item
        int cur = seg[i], pos = 1;
        team_sum[0] = w[i];
        ++i;
        while (i < n) {
            const bool new_run = seg[i] != cur;
            const double c2 = new_run ? closed + run_time(run_max, run_work) : closed;
            const int p2 = new_run ? 0 : pos;
            const double t2 = (new_run ? 0.0 : team_sum[p2 % teams]) + w[i];
            const double m2 = new_run ? t2 : (run_max > t2 ? run_max : t2);
            const double k2 = (new_run ? 0.0 : run_work) + w[i];
            if (c2 + run_time(m2, k2) > bound) break;
            if (new_run) { for (int t = 0; t < teams; ++t) team_sum[t] = 0.0; cur = seg[i]; }
            closed = c2; run_max = m2; run_work = k2; team_sum[p2 % teams] = t2; pos = p2 + 1;
            ++i;
        }
        return i;
    };
    auto blocks_needed = [&](double bound) {
        int64_t blocks = 0;
        for (int64_t i = 0; i < n; i = reach(i, bound)) ++blocks;
        return blocks;
    };
    double lo = 0.0, hi = 0.0;
    for (int64_t i = 0; i < n; ++i) hi += w[i] + run_cost;
    for (int it = 0; it < 60; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (blocks_needed(mid) <= max_blocks) hi = mid; else lo = mid;
    }
    // Within the bound found, spread the items over ALL the blocks: the greedy fill would leave the last
    // blocks empty, and a block with less work is never slower.  need[i] = blocks a greedy fill needs for
    // the items i .. n-1; a cut at i before block b is admissible if the rest still fits the blocks left.
    const int64_t blocks = max_blocks < n ? max_blocks : n;
    int32_t* need = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n + 1));
    double* pre = (double*)malloc(sizeof(double) * (size_t)(n + 1));
    if (!need || !pre) { free(need); free(pre); return -1; }
    {   // backwards: need[i] = 1 + need[reach(i)], computed with a moving window of block starts
        need[n] = 0;
        for (int64_t i = n - 1; i >= 0; --i) need[i] = 1 + need[reach(i, hi)];
        pre[0] = 0.0;
        for (int64_t i = 0; i < n; ++i) pre[i + 1] = pre[i] + w[i];
    }
    int64_t at = 0;
    for (int64_t b = 0; b < blocks; ++b) {
        part[b] = (int32_t)at;
        if (at >= n) continue;
        const int64_t far = reach(at, hi);                  // the block may end anywhere in (at, far]
        const double target = pre[n] * (double)(b + 1) / (double)blocks;
        int64_t end = at + 1;
        while (end < far && pre[end] < target) ++end;       // proportional share of the work ...
        while (end < far && need[end] > blocks - b - 1) ++end;   // ... unless the rest would not fit
        if (n - end < blocks - b - 1) end = n - (blocks - b - 1) > at ? n - (blocks - b - 1) : at + 1;   // leave an item for every later block
        at = end;
    }
    for (int64_t b = blocks; b <= max_blocks; ++b) part[b] = (int32_t)n;
    part[blocks] = (int32_t)n;
    free(need); free(pre);
    return (int)blocks;
}

extern "C" int co3_balanced_split(const double* cost, const int32_t* seg, int64_t n, int32_t teams, int32_t max_blocks,
                                  int32_t* part) {
    return co3_host_balanced_split(cost, seg, n, teams, max_blocks, 0.08, part);
}

extern "C" uint64_t co3_model_checksum(co3_format fmt) {
    if (!co3_host_fmt_ok(fmt)) return 0;
    const uint32_t* t = co3_host_weight_table(fmt.exp_bits, fmt.mant_bits);
    if (!t) return 0;
    const size_t n = (size_t)CO3_NIBETA * CO3_NIR * ((size_t)1 << (fmt.exp_bits + fmt.mant_bits));
    uint64_t h = 0xcbf29ce484222325ull;              // FNV-1a over the table's words, byte by byte, low byte first
    for (size_t i = 0; i < n; ++i)
        for (int b = 0; b < 4; ++b) { h ^= (t[i] >> (8 * b)) & 0xFFu; h *= 0x100000001b3ull; }
    return h ? h : 1;
}

extern "C" int64_t co3_partition(int64_t d, int32_t n_segments, const int64_t* seg_offsets,
                                 int32_t* chunk_seg, int64_t* chunk_start, int64_t* chunk_end,
                                 int64_t* sub_base, int64_t* n_sub) {
    const int64_t one_seg[2] = {0, d};
    if (!seg_offsets) { seg_offsets = one_seg; n_segments = 1; }
    if (d < 1 || n_segments < 1 || seg_offsets[0] != 0 || seg_offsets[n_segments] != d) return CO3_EINVAL;
    int64_t nc = 0, ns = 0;
    for (int l = 0; l < n_segments; ++l) {
        int64_t lo = seg_offsets[l], hi = seg_offsets[l + 1];
        if (hi < lo) return CO3_EINVAL;
        while (lo < hi) {
            int64_t cut = (lo / CO3_TILE + 1) * CO3_TILE;
            if (cut > hi) cut = hi;
            if (chunk_seg) chunk_seg[nc] = l;
            if (chunk_start) chunk_start[nc] = lo;
            if (chunk_end) chunk_end[nc] = cut;
            if (sub_base) sub_base[nc] = ns;
            ns += (cut - 1) / CO3_SUB - lo / CO3_SUB + 1;
            ++nc;
            lo = cut;
        }
    }
    if (n_sub) *n_sub = ns;
    return nc;
}
