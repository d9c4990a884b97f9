/*
 * CO3 oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU statement of the per-iteration CO3 gradient pipeline of
 * "Convert, compress, correct: three steps toward communication-efficient DNN training"
 * (Algorithm 1 lines 8-10 at the user, lines 13-14 at the parameter server; Sec. III (i)-(iii);
 * Eq. "exp bias"; Eq. "approximate").  It exists so that the CUDA library can be checked
 * against something that can be compared with the paper by eye.  It shares no code, header,
 * table or constant generator with the CUDA library, and only tests, the smoke check and the
 * CPU-baseline leg of the benchmark may call it.
 *
 * Every step is written in the order and notation of the paper; where the paper is silent the
 * reading taken is stated at the function that implements it.  Floating point: the values that
 * the method itself carries (gradient, memory, quantised gradient) are fp32 as in the paper's
 * setting; everything derived (moments, fit, model probabilities) is fp64, with sums held in a
 * long double accumulator.
 *
 * Build: gcc -O2 -ffp-contract=off -shared -fPIC co3_oracle.c -lm   (no FMA contraction:
 * "a = g + gamma*m" must round twice, Algorithm 1 line 8).
 *
 * Parity pins (tests, CPU only): grid representability and the worked fp4 grid, brute-force
 * nearest-point search, the telescoping identity q + m' = g + gamma*m in exact arithmetic,
 * closed forms of the GenNorm moment ratio, closed forms of the GenNorm CDF at beta = 1/2, 1, 2,
 * re-optimisation of the fp4 scale against the bias polynomial, Kraft equality, prefix-freeness
 * and brute-force optimality of the code, decode(encode(x)) == x, U = 1 average == q.
 * Parity unpinned (the paper prints no number for them): optimality of the bias for formats
 * other than fp4, handling of non-finite inputs, compression ratio, accuracy.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define CO3O_TILE 4096   /* chunk grid: chunks are cut at multiples of 4096 elements ...      */
#define CO3O_SUB 128     /* ... and sub-chunks at multiples of 128 elements of the user's row */
#define CO3O_MAXLEN 16   /* longest codeword                                                  */
#define CO3O_WSCALE 1048576.0 /* W = 2^20: probability -> integer weight                      */

#define CO3O_OK 0
#define CO3O_EINVAL (-1)
#define CO3O_ECAPACITY (-4)
#define CO3O_ECORRUPT (-5)

/* ------------------------------------------------------------------------------------------
 * Format: 1 sign bit, E exponent bits, M mantissa bits (Sec. III (i)).  Reading: IEEE-like grid
 * with gradual underflow (zero is a grid point), standard exponent bias 2^(E-1)-1 shifted by the
 * integer exponent bias b of Eq. "exp bias", no Inf/NaN codes.  Magnitude code j = (e << M) | f.
 * Grid value  v(s, j) = (-1)^s * K(j) * 2^lambda,  lambda = b + c_F,  c_F = 1 - bias_F - M,
 * which is Eq. "exp bias"'s  c_sgn * c_mant * 2^(c_exp + b)  with c_mant = 1.f (0.f when e = 0)
 * and c_exp = max(e, 1) - bias_F.
 * ------------------------------------------------------------------------------------------ */
static int fmt_ok(int E, int M) { return E >= 1 && E <= 4 && M >= 1 && E + M <= 7; }

int co3o_num_mag(int E, int M) { return fmt_ok(E, M) ? 1 << (E + M) : 0; }

int64_t co3o_K(int E, int M, int j) {
    (void)E;
    int e = j >> M, f = j & ((1 << M) - 1);
    if (e == 0) return f;                       /* subnormal: 0.f * 2^(1 - bias_F)            */
    return (int64_t)((1 << M) + f) << (e - 1);  /* normal:    1.f * 2^(e - bias_F)            */
}

static int bias_F(int E) { return (1 << (E - 1)) - 1; }

int co3o_cF(int E, int M) { return 1 - bias_F(E) - M; }

int64_t co3o_Kmax(int E, int M) { return co3o_K(E, M, (1 << (E + M)) - 1); }

/* Integer bias range: every grid value must be a normal fp32 number or zero.
 * lambda >= -120, and the largest grid value K_max * 2^lambda < 2^100.                        */
int co3o_b_lo(int E, int M) { return -120 - co3o_cF(E, M); }
int co3o_b_hi(int E, int M) {
    int64_t km = co3o_Kmax(E, M);
    int bl = 0;
    while ((km >> bl) != 0) bl++;               /* K_max < 2^bl */
    return (100 - bl) - co3o_cF(E, M);
}

/* v(s, j) for symbol byte sym = (s << (E+M)) | j, as an fp32 number. */
float co3o_grid_value(int E, int M, int b, int sym) {
    int nm = E + M;
    int s = (sym >> nm) & 1, j = sym & ((1 << nm) - 1);
    double v = ldexp((double)co3o_K(E, M, j), b + co3o_cF(E, M));
    return (float)(s ? -v : v);
}

/* Round a non-negative real that is exactly representable in double to the nearest integer,
 * ties to the even integer. */
static double rne(double y) {
    double r = floor(y), d = y - r;
    if (d > 0.5 || (d == 0.5 && fmod(r, 2.0) != 0.0)) r += 1.0;
    return r;
}

/* Q_fp: nearest grid point to a (Sec. III (i), "closest quantization representative"), ties to
 * the even magnitude code, saturating at +-K_max after rounding.  Returns the symbol byte and
 * the integer magnitude k with q = +-k * 2^lambda.  a must be finite. */
static int quantize(float a, int E, int M, int lambda, int64_t* k_out) {
    double y = ldexp(fabs((double)a), -lambda);         /* |a| / 2^lambda, exact               */
    double k;
    if (y < ldexp(1.0, M + 1)) {
        k = rne(y);                                     /* quantum 1 up to the first binade    */
    } else {
        int ex;
        (void)frexp(y, &ex);                            /* y in [2^(ex-1), 2^ex)               */
        double u = ldexp(1.0, (ex - 1) - M);            /* quantum of y's binade               */
        k = u * rne(y / u);                             /* may carry into the next binade      */
    }
    double kmax = (double)co3o_Kmax(E, M);
    if (k > kmax) k = kmax;
    int64_t ki = (int64_t)k;
    int j;                                              /* j = K^-1(k)                         */
    if (ki < ((int64_t)1 << (M + 1))) {
        j = (int)ki;                                    /* e = 0: j = f;  e = 1: j = 2^M + f   */
    } else {
        int p = 0;
        while ((ki >> (p + 1)) != 0) p++;               /* ki in [2^p, 2^(p+1))                */
        int f = (int)(ki >> (p - M)) - (1 << M);
        j = ((p - M + 1) << M) | f;
    }
    if (co3o_K(E, M, j) != ki) abort();                 /* k must be a grid magnitude          */
    int s = (a < 0.0f && ki > 0) ? 1 : 0;               /* -0 is never emitted                 */
    *k_out = ki;
    return (s << (E + M)) | j;
}

int co3o_quantize_one(float a, int E, int M, int b, float* q) {
    int64_t k;
    int sym = quantize(a, E, M, b + co3o_cF(E, M), &k);
    *q = co3o_grid_value(E, M, b, sym);
    return sym;
}

/* ------------------------------------------------------------------------------------------
 * Moments of a = g + gamma*m over one segment [lo, hi) of every user's row, pooled over users
 * (the model is fitted to g_t + gamma m_{t-1}, Sec. IV-B "Huffman coding"; one code per layer
 * shared by all users, Sec. III (ii)).  Non-finite a are counted and left out.
 * ------------------------------------------------------------------------------------------ */
static float ef_add(float g, float m, float gamma) {
    volatile float gm = gamma * m;      /* fl32(gamma * m) */
    volatile float a = g + gm;          /* fl32(g + .)     */
    return a;
}

void co3o_stats(const float* g, const float* m, int U, int64_t ld, int64_t lo, int64_t hi,
                float gamma, double* N, double* S1, double* S2, int64_t* nonfinite) {
    long double s1 = 0.0L, s2 = 0.0L;
    int64_t n = 0, nf = 0;
    for (int u = 0; u < U; u++)
        for (int64_t i = lo; i < hi; i++) {
            float a = ef_add(g[u * ld + i], m[u * ld + i], gamma);
            if (!isfinite(a)) { nf++; continue; }
            double ad = fabs((double)a);
            s1 += ad;
            s2 += ad * ad;                              /* exact in double */
            n++;
        }
    *N = (double)n; *S1 = (double)s1; *S2 = (double)s2; *nonfinite = nf;
}

/* Algorithm 1 lines 8 and 10 for one segment and all users:
 *   a = g + gamma m;  ghat = Q_fp(a);  m <- a - ghat  (= gamma m + g - ghat).
 * Writes the symbol bytes (row pitch sld), updates m in place, adds to hist[2^B] and returns
 * the moments of a as co3o_stats does.  Non-finite a: counted, coded as +0, m reset to 0. */
void co3o_convert(const float* g, float* m, uint8_t* sym, int U, int64_t ld, int64_t sld,
                  int64_t lo, int64_t hi, float gamma, int E, int M, int b, uint64_t* hist,
                  double* N, double* S1, double* S2, int64_t* nonfinite) {
    int lambda = b + co3o_cF(E, M);
    long double s1 = 0.0L, s2 = 0.0L;
    int64_t n = 0, nf = 0;
    for (int u = 0; u < U; u++)
        for (int64_t i = lo; i < hi; i++) {
            float a = ef_add(g[u * ld + i], m[u * ld + i], gamma);
            if (!isfinite(a)) {
                nf++;
                sym[u * sld + i] = 0;
                hist[0]++;
                m[u * ld + i] = 0.0f;
                continue;
            }
            double ad = fabs((double)a);
            s1 += ad; s2 += ad * ad; n++;
            int64_t k;
            int sy = quantize(a, E, M, lambda, &k);
            double qd = ldexp((double)k, lambda);
            volatile float q = (float)((sy >> (E + M)) ? -qd : qd);   /* exact */
            volatile float r = a - q;                                 /* fl32(a - q) */
            m[u * ld + i] = r;
            sym[u * sld + i] = (uint8_t)sy;
            hist[sy]++;
        }
    *N = (double)n; *S1 = (double)s1; *S2 = (double)s2; *nonfinite = nf;
}

/* ------------------------------------------------------------------------------------------
 * GenNorm fit by moment matching (reading of "best-fit"): zero-location density
 * f(x) ~ exp(-(|x|/alpha)^beta);  E|X| = alpha G(2/b)/G(1/b),  E X^2 = alpha^2 G(3/b)/G(1/b),
 * so  E X^2 / (E|X|)^2 = R(beta) = G(1/b) G(3/b) / G(2/b)^2, strictly decreasing in beta.
 * beta is clamped to [0.3, 2.0] first and alpha is then taken from E|X|.
 * ------------------------------------------------------------------------------------------ */
double co3o_logR(double beta) {
    return lgamma(1.0 / beta) + lgamma(3.0 / beta) - 2.0 * lgamma(2.0 / beta);
}

void co3o_fit(double N, double S1, double S2, double* beta, double* alpha) {
    if (!(N > 0.0) || !(S1 > 0.0)) { *beta = 1.0; *alpha = 0.0; return; }
    double target = log(N) + log(S2) - 2.0 * log(S1);   /* log rho */
    double lo = 0.3, hi = 2.0, b;
    if (target >= co3o_logR(lo)) b = lo;
    else if (target <= co3o_logR(hi)) b = hi;
    else {
        for (int it = 0; it < 200 && (hi - lo) > 1e-15 * hi; it++) {
            double mid = 0.5 * (lo + hi);
            if (co3o_logR(mid) > target) lo = mid; else hi = mid;   /* R decreasing */
        }
        b = 0.5 * (lo + hi);
    }
    *beta = b;
    *alpha = (S1 / N) * exp(lgamma(1.0 / b) - lgamma(2.0 / b));
}

/* Eq. "approximate": polynomial in the shape parameter. */
double co3o_poly(double beta) {
    double b2 = beta * beta;
    return 0.46 - 2.85 * beta + 5.37 * b2 - 2.85 * b2 * beta + 0.52 * b2 * b2;
}

/* Exponent bias.  Reading of Eq. "approximate": the right-hand side is the scalar that multiplies
 * the gradient before a standard-bias conversion, with sigma the GenNorm scale alpha; as an
 * exponent bias that is b_real = log2(alpha) - log2(P(beta)).  The grid must be representable,
 * so the nearest integer (half up) is used, clamped to the admissible range. */
int co3o_bias(double beta, double alpha, int E, int M) {
    int lo = co3o_b_lo(E, M), hi = co3o_b_hi(E, M);
    if (!(alpha > 0.0)) return lo;
    double br = log2(alpha) - log2(co3o_poly(beta));
    double bf = floor(br + 0.5);
    if (bf < (double)lo) return lo;
    if (bf > (double)hi) return hi;
    return (int)bf;
}

/* Side information that names the code model: shape and scale (relative to the bias actually
 * used) on a grid of 1/8 in log2, so that user and PS build the same code from three small
 * integers per segment. */
void co3o_header(double beta, double alpha, int b, int* ibeta, int* ir) {
    double x = floor(8.0 * log2(beta) + 0.5);
    if (x < -14.0) x = -14.0;
    if (x > 8.0) x = 8.0;
    *ibeta = (int)x;
    if (!(alpha > 0.0)) { *ir = -96; return; }
    double y = floor(8.0 * (log2(alpha) - (double)b) + 0.5);
    if (y < -96.0) y = -96.0;
    if (y > 31.0) y = 31.0;
    *ir = (int)y;
}

/* ------------------------------------------------------------------------------------------
 * Regularised lower incomplete gamma P(a, x): power series for x < a + 1, continued fraction
 * (modified Lentz) for the complement otherwise.  For zero-location GenNorm,
 * Pr(|X| <= t) = P(1/beta, (t/alpha)^beta).
 * ------------------------------------------------------------------------------------------ */
double co3o_gammainc(double a, double x) {
    if (!(x > 0.0)) return 0.0;
    if (isinf(x)) return 1.0;
    double lead = a * log(x) - x - lgamma(a);           /* log( x^a e^-x / Gamma(a) ) */
    if (x < a + 1.0) {
        double term = 1.0 / a, sum = term, ap = a;
        for (int n = 0; n < 100000; n++) {
            ap += 1.0;
            term *= x / ap;
            sum += term;
            if (fabs(term) < fabs(sum) * 1e-17) break;
        }
        double p = sum * exp(lead);
        return p > 1.0 ? 1.0 : p;
    }
    /* Q(a,x) = e^lead / (x+1-a- 1(1-a)/(x+3-a- 2(2-a)/(x+5-a- ...))) */
    const double tiny = 1e-300;
    double bb = x + 1.0 - a, c = 1.0 / tiny, d = 1.0 / bb, h = d;
    for (int i = 1; i < 100000; i++) {
        double an = -(double)i * ((double)i - a);
        bb += 2.0;
        d = an * d + bb; if (fabs(d) < tiny) d = tiny;
        c = bb + an / c; if (fabs(c) < tiny) c = tiny;
        d = 1.0 / d;
        double del = d * c;
        h *= del;
        if (fabs(del - 1.0) < 1e-16) break;
    }
    double q = exp(lead) * h;
    if (q < 0.0) q = 0.0;
    if (q > 1.0) q = 1.0;
    return 1.0 - q;
}

/* ------------------------------------------------------------------------------------------
 * The quantity the exponent bias is meant to minimise (Eq. "exp bias", L2 reading): the expected
 * squared conversion error of X ~ GenNorm(alpha, beta), here divided by alpha^2 and evaluated on the
 * header grid: beta = 2^(ibeta/8), log2(alpha) - b = ir/8.  In units of alpha the grid values are
 * v_j = K(j) u with u = 2^(c_F - ir/8), the cells end at the midpoints t_j = (v_j + v_(j+1)) / 2 (the
 * last one at infinity: saturation), and with z = (x/alpha)^beta
 *   int_0^t (x/alpha)^k dF = Gamma((k+1)/beta) / Gamma(1/beta) * P((k+1)/beta, t^beta),
 * so each cell contributes m2 - 2 v m1 + v^2 m0 from differences of three incomplete gammas.
 * ------------------------------------------------------------------------------------------ */
double co3o_distortion(int E, int M, int ibeta, int ir) {
    if (!fmt_ok(E, M)) return -1.0;
    int J = 1 << (E + M);
    double beta = exp2((double)ibeta / 8.0);
    double u = exp2((double)co3o_cF(E, M) - (double)ir / 8.0);
    double a0 = 1.0 / beta, a1 = 2.0 / beta, a2 = 3.0 / beta;
    double c1 = exp(lgamma(a1) - lgamma(a0)), c2 = exp(lgamma(a2) - lgamma(a0));
    double p0 = 0.0, p1 = 0.0, p2 = 0.0, total = 0.0;
    for (int j = 0; j < J; j++) {
        double q0 = 1.0, q1 = 1.0, q2 = 1.0;
        if (j < J - 1) {
            double t = 0.5 * (double)(co3o_K(E, M, j) + co3o_K(E, M, j + 1)) * u;
            double z = pow(t, beta);
            q0 = co3o_gammainc(a0, z); q1 = co3o_gammainc(a1, z); q2 = co3o_gammainc(a2, z);
        }
        double v = (double)co3o_K(E, M, j) * u;
        total += c2 * (q2 - p2) - 2.0 * v * c1 * (q1 - p1) + v * v * (q0 - p0);
        p0 = q0; p1 = q1; p2 = q2;
    }
    return total;
}

/* Bias rule "optimal": the integer b that minimises that distortion.  Shifting b by one moves ir by
 * eight, so for a shape index ibeta and a residue rho = round(8 log2 alpha) mod 8 the choice is the
 * best ir among those congruent to rho: a table of 23 x 8 entries per format (first minimum in
 * ascending ir, i.e. the larger bias on an exact tie). */
void co3o_bias_opt_table(int E, int M, int16_t* tab) {
    for (int ib = -14; ib <= 8; ib++)
        for (int rho = 0; rho < 8; rho++) {
            int best = 0, have = 0;
            double dbest = 0.0;
            for (int ir = -96; ir <= 31; ir++) {
                if ((((ir % 8) + 8) % 8) != rho) continue;
                double dd = co3o_distortion(E, M, ib, ir);
                if (!have || dd < dbest) { have = 1; dbest = dd; best = ir; }
            }
            tab[(ib + 14) * 8 + rho] = (int16_t)best;
        }
}

int co3o_bias_opt(double beta, double alpha, int E, int M, const int16_t* tab) {
    int lo = co3o_b_lo(E, M), hi = co3o_b_hi(E, M);
    if (!(alpha > 0.0)) return lo;
    double x = floor(8.0 * log2(beta) + 0.5);
    if (x < -14.0) x = -14.0;
    if (x > 8.0) x = 8.0;
    double t8 = floor(8.0 * log2(alpha) + 0.5);
    if (t8 < -16000.0) return lo;
    if (t8 > 16000.0) return hi;
    int t = (int)t8, rho = ((t % 8) + 8) % 8;
    int b = (t - (int)tab[((int)x + 14) * 8 + rho]) / 8;      /* exact: same residue */
    return b < lo ? lo : (b > hi ? hi : b);
}

/* Integer symbol weights of the quantised GenNorm model (Sec. IV-B "Huffman coding": the
 * converted samples follow the quantised GenNorm distribution) for header indices (ibeta, ir).
 * Cell edges are the midpoints between neighbouring grid magnitudes, in units of alpha.
 * w has 2^(1+E+M) entries indexed by symbol byte. */
int co3o_model_weights(int E, int M, int ibeta, int ir, uint32_t* w) {
    if (!fmt_ok(E, M) || ibeta < -14 || ibeta > 8 || ir < -96 || ir > 31) return CO3O_EINVAL;
    int J = 1 << (E + M);
    double beta_q = exp2((double)ibeta / 8.0), r_q = (double)ir / 8.0;
    double unit = exp2((double)co3o_cF(E, M) - r_q);    /* grid quantum / alpha */
    double Fprev = 0.0;
    for (int j = 0; j < J; j++) {
        double F = 1.0;
        if (j < J - 1) {
            double tau = 0.5 * (double)(co3o_K(E, M, j) + co3o_K(E, M, j + 1)) * unit;
            F = co3o_gammainc(1.0 / beta_q, pow(tau, beta_q));
        }
        double mass = F - Fprev;
        Fprev = F;
        if (j == 0) {
            double x = floor(CO3O_WSCALE * mass + 0.5);
            w[0] = x < 1.0 ? 1u : (uint32_t)x;          /* +0 takes the whole central cell */
            w[J] = 1u;                                  /* -0 is never emitted             */
        } else {
            double x = floor(CO3O_WSCALE * mass / 2.0 + 0.5);
            uint32_t wi = x < 1.0 ? 1u : (uint32_t)x;
            w[j] = wi;
            w[J + j] = wi;
        }
    }
    return CO3O_OK;
}

/* ------------------------------------------------------------------------------------------
 * Huffman code lengths (Sec. III (ii), element-wise Huffman coding) over the whole alphabet.
 * Deterministic form: leaves sorted by (weight, symbol); two queues (sorted leaves, internal
 * nodes in creation order); on equal weights the leaf is taken first.  Depth limit 16: weights
 * are raised to a floor f = 1, 2, 4, ... until the Huffman code of the floored weights has no
 * codeword longer than 16 (it is still a Huffman code, of the floored weights).
 * ------------------------------------------------------------------------------------------ */
static int huffman_once(const uint64_t* wp, int n, uint8_t* len) {
    int* order = (int*)malloc(sizeof(int) * (size_t)n);
    for (int i = 0; i < n; i++) order[i] = i;
    for (int i = 1; i < n; i++) {                       /* insertion sort by (weight, symbol) */
        int s = order[i], k = i - 1;
        while (k >= 0 && (wp[order[k]] > wp[s] || (wp[order[k]] == wp[s] && order[k] > s))) {
            order[k + 1] = order[k];
            k--;
        }
        order[k + 1] = s;
    }
    uint64_t* iw = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)n);
    int* parent = (int*)malloc(sizeof(int) * (size_t)(2 * n));
    int* depth = (int*)malloc(sizeof(int) * (size_t)(2 * n));
    int i = 0, j = 0;                                   /* heads of the two queues */
    for (int k = 0; k < n - 1; k++) {
        uint64_t sum = 0;
        for (int t = 0; t < 2; t++) {
            int node;
            if (i < n && (j >= k || wp[order[i]] <= iw[j])) { node = i; sum += wp[order[i]]; i++; }
            else { node = n + j; sum += iw[j]; j++; }
            parent[node] = n + k;
        }
        iw[k] = sum;
    }
    int root = n + (n - 2), maxlen = 0;
    depth[root] = 0;
    for (int k = n - 3; k >= 0; k--) depth[n + k] = depth[parent[n + k]] + 1;
    for (int p = 0; p < n; p++) {
        int dl = depth[parent[p]] + 1;
        if (dl > maxlen) maxlen = dl;
        len[order[p]] = (uint8_t)(dl > 255 ? 255 : dl);
    }
    free(order); free(iw); free(parent); free(depth);
    return maxlen;
}

int co3o_huffman(const uint32_t* w, int n, uint8_t* len, uint32_t* floor_used) {
    if (n < 2) return CO3O_EINVAL;
    uint64_t* wp = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)n);
    uint64_t f = 1;
    for (;;) {
        for (int s = 0; s < n; s++) wp[s] = w[s] > f ? w[s] : f;
        if (huffman_once(wp, n, len) <= CO3O_MAXLEN) break;
        f *= 2;
    }
    free(wp);
    if (floor_used) *floor_used = (uint32_t)f;
    return CO3O_OK;
}

/* Empirical-histogram variant: the code of a layer is the Huffman code of the symbol counts of
 * this iteration (pooled over users), built exactly like the model code (full alphabet, floor 1 for
 * symbols that did not occur, same tie-breaks and depth limit).  Counts are brought into 32 bits by
 * dropping the k low bits that make the layer's total fit below 2^31. */
int co3o_huffman_counts(const uint64_t* counts, int n, uint8_t* len, uint32_t* floor_used) {
    if (n < 2 || n > 256) return CO3O_EINVAL;
    uint64_t tot = 0;
    for (int s = 0; s < n; s++) tot += counts[s];
    int k = 0;
    while ((tot >> k) >= ((uint64_t)1 << 31)) k++;
    uint32_t w[256];
    for (int s = 0; s < n; s++) w[s] = (uint32_t)(counts[s] >> k);
    return co3o_huffman(w, n, len, floor_used);
}

/* Canonical codewords: symbols ordered by (length, symbol); code values as integers whose most
 * significant of `len` bits is the root branch. */
void co3o_canonical(const uint8_t* len, int n, uint32_t* code) {
    uint32_t count[CO3O_MAXLEN + 2] = {0}, first[CO3O_MAXLEN + 2] = {0};
    for (int s = 0; s < n; s++) count[len[s]]++;
    uint32_t c = 0;
    for (int L = 1; L <= CO3O_MAXLEN; L++) { first[L] = c; c = (c + count[L]) << 1; }
    uint32_t next[CO3O_MAXLEN + 2];
    memcpy(next, first, sizeof(next));
    for (int s = 0; s < n; s++) code[s] = next[len[s]]++;
}

/* ------------------------------------------------------------------------------------------
 * Container.  A user's row of d symbols is cut into chunks at every multiple of 4096 elements
 * and at every segment boundary (a chunk never spans two segments, so it has one code), and
 * every chunk into sub-chunks at multiples of 128 elements.  Chunk c of user u occupies the
 * 32-bit words [chunk_off[c], chunk_off[c+1]) of the user's payload; a chunk's word count is
 * its bit count rounded up to a multiple of 128 bits.  Inside a chunk codewords follow one
 * another with no gaps; stream bit p is bit (p & 31) of word (p >> 5); a codeword's root bit
 * comes first; pad bits are zero.  sub_bits[k] is the bit length of sub-chunk k.
 * ------------------------------------------------------------------------------------------ */
int64_t co3o_partition(int64_t d, int S, const int64_t* off, int32_t* chunk_seg,
                       int64_t* chunk_start, int64_t* chunk_end, int64_t* sub_base,
                       int64_t* n_sub_out) {
    if (S < 1 || off[0] != 0 || off[S] != d) return CO3O_EINVAL;
    int64_t nc = 0, ns = 0;
    for (int l = 0; l < S; l++) {
        if (off[l + 1] < off[l]) return CO3O_EINVAL;
        int64_t start = off[l];
        while (start < off[l + 1]) {
            int64_t end = (start / CO3O_TILE + 1) * CO3O_TILE;
            if (end > off[l + 1]) end = off[l + 1];
            if (chunk_seg) {
                chunk_seg[nc] = l; chunk_start[nc] = start; chunk_end[nc] = end; sub_base[nc] = ns;
            }
            ns += (end + CO3O_SUB - 1) / CO3O_SUB - start / CO3O_SUB;
            nc++;
            start = end;
        }
    }
    if (n_sub_out) *n_sub_out = ns;
    return nc;
}

static void put_bit(uint32_t* words, int64_t p, int bit) {
    if (bit) words[p >> 5] |= (uint32_t)1 << (p & 31);
}
static int get_bit(const uint32_t* words, int64_t p) {
    return (int)((words[p >> 5] >> (p & 31)) & 1u);
}

/* h_Hf for one user (Algorithm 1 line 9).  len/code are [S][2^B].  Returns CO3O_ECAPACITY (and
 * writes no payload) when the payload would not fit cap_words; chunk_off, sub_bits and
 * user_bits are written either way. */
int co3o_encode_user(const uint8_t* sym, int64_t n_chunks, const int32_t* chunk_seg,
                     const int64_t* chunk_start, const int64_t* chunk_end, const int64_t* sub_base,
                     int nsym, const uint8_t* len, const uint32_t* code, uint32_t* payload,
                     int64_t cap_words, uint16_t* sub_bits, uint32_t* chunk_off,
                     uint64_t* user_bits) {
    uint64_t total_bits = 0;
    int64_t woff = 0;
    for (int64_t c = 0; c < n_chunks; c++) {            /* sizes first */
        const uint8_t* L = len + (size_t)chunk_seg[c] * (size_t)nsym;
        int64_t bits = 0, k = sub_base[c], sb = 0;
        for (int64_t i = chunk_start[c]; i < chunk_end[c]; i++) {
            sb += L[sym[i]];
            if ((i + 1) % CO3O_SUB == 0 || i + 1 == chunk_end[c]) {
                sub_bits[k++] = (uint16_t)sb; bits += sb; sb = 0;
            }
        }
        chunk_off[c] = (uint32_t)woff;
        woff += 4 * ((bits + 127) / 128);
        total_bits += (uint64_t)bits;
    }
    chunk_off[n_chunks] = (uint32_t)woff;
    *user_bits = total_bits;
    if (woff > cap_words) return CO3O_ECAPACITY;
    memset(payload, 0, sizeof(uint32_t) * (size_t)woff);
    for (int64_t c = 0; c < n_chunks; c++) {
        const uint8_t* L = len + (size_t)chunk_seg[c] * (size_t)nsym;
        const uint32_t* C = code + (size_t)chunk_seg[c] * (size_t)nsym;
        uint32_t* words = payload + chunk_off[c];
        int64_t p = 0;
        for (int64_t i = chunk_start[c]; i < chunk_end[c]; i++) {
            int l = L[sym[i]];
            uint32_t cw = C[sym[i]];
            for (int bpos = l - 1; bpos >= 0; bpos--) put_bit(words, p++, (int)((cw >> bpos) & 1u));
        }
    }
    return CO3O_OK;
}

/* Algorithm 1 lines 13-14 up to the model update: rebuild every segment's code from the header
 * alone, decode every user's stream and average,  avg = (1/U) sum_u ghat^(u)  (Eq. "aggregate").
 * The sum is taken over the integer magnitudes (exact) and scaled once:
 * avg = fl32( fl32(K_sum) * 2^lambda ) / fl32(U).
 * hdr is [S][3] int32: (b, ibeta, ir).  With lens_in ([S][2^B] code lengths, the side information
 * of the empirical-histogram code) the codes are the canonical codes of those lengths instead.
 * Returns CO3O_ECORRUPT if a sub-chunk does not decode to exactly its recorded bit length, a chunk
 * runs past its words, or given lengths are not those of a complete prefix code. */
int co3o_decode_aggregate(const uint32_t* payload, int64_t cap_words, const uint16_t* sub_bits,
                          int64_t n_sub, const uint32_t* chunk_off, int U, int64_t n_chunks,
                          const int32_t* chunk_seg, const int64_t* chunk_start,
                          const int64_t* chunk_end, const int64_t* sub_base, int S,
                          const int32_t* hdr, int E, int M, float* avg, uint8_t* sym_out,
                          int64_t sld, const uint8_t* lens_in) {
    int nsym = 1 << (1 + E + M), nm = E + M;
    uint8_t* len = (uint8_t*)malloc((size_t)S * (size_t)nsym);
    uint32_t* code = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)S * (size_t)nsym);
    uint32_t* w = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)nsym);
    /* canonical decoding tables per segment: for every length the first code value, the number
     * of codewords, and where that length's symbols start in the (length, symbol) ordering */
    const int NL = CO3O_MAXLEN + 2;
    uint32_t* first = (uint32_t*)calloc((size_t)S * (size_t)NL, sizeof(uint32_t));
    uint32_t* count = (uint32_t*)calloc((size_t)S * (size_t)NL, sizeof(uint32_t));
    uint32_t* start = (uint32_t*)calloc((size_t)S * (size_t)NL, sizeof(uint32_t));
    int* sorted = (int*)malloc(sizeof(int) * (size_t)S * (size_t)nsym);
    int rc = CO3O_OK;
    for (int l = 0; l < S && rc == CO3O_OK; l++) {
        uint8_t* L = len + (size_t)l * nsym;
        uint32_t* C = code + (size_t)l * nsym;
        if (lens_in) {                                  /* empirical code: the lengths are side information */
            double kraft = 0.0;
            for (int s = 0; s < nsym; s++) {
                L[s] = lens_in[(size_t)l * nsym + s];
                if (L[s] < 1 || L[s] > CO3O_MAXLEN) { rc = CO3O_ECORRUPT; break; }
                kraft += ldexp(1.0, -(int)L[s]);
            }
            if (rc == CO3O_OK && kraft != 1.0) rc = CO3O_ECORRUPT;
            if (rc != CO3O_OK) break;
        } else {
            rc = co3o_model_weights(E, M, hdr[3 * l + 1], hdr[3 * l + 2], w);
            if (rc != CO3O_OK) break;
            co3o_huffman(w, nsym, L, NULL);
        }
        co3o_canonical(L, nsym, C);
        uint32_t *fi = first + (size_t)l * NL, *cn = count + (size_t)l * NL, *st = start + (size_t)l * NL;
        for (int s = 0; s < nsym; s++) cn[L[s]]++;
        uint32_t acc = 0;
        for (int ll = 1; ll <= CO3O_MAXLEN; ll++) { st[ll] = acc; acc += cn[ll]; }
        for (int ll = 1; ll <= CO3O_MAXLEN; ll++) fi[ll] = 0xFFFFFFFFu;
        for (int s = 0; s < nsym; s++) if (C[s] < fi[L[s]]) fi[L[s]] = C[s];
        for (int s = 0; s < nsym; s++) sorted[(size_t)l * nsym + st[L[s]] + (C[s] - fi[L[s]])] = s;
    }
    int64_t* ksum = (int64_t*)malloc(sizeof(int64_t) * CO3O_TILE);
    for (int64_t c = 0; c < n_chunks && rc == CO3O_OK; c++) {
        int l = chunk_seg[c];
        const uint32_t *fi = first + (size_t)l * NL, *cn = count + (size_t)l * NL, *st = start + (size_t)l * NL;
        const int* so = sorted + (size_t)l * nsym;
        int64_t n = chunk_end[c] - chunk_start[c];
        memset(ksum, 0, sizeof(int64_t) * (size_t)n);
        for (int u = 0; u < U && rc == CO3O_OK; u++) {
            const uint32_t* co = chunk_off + (size_t)u * (size_t)(n_chunks + 1);
            const uint32_t* words = payload + (size_t)u * (size_t)cap_words + co[c];
            int64_t avail = 32 * ((int64_t)co[c + 1] - (int64_t)co[c]);
            const uint16_t* sb = sub_bits + (size_t)u * (size_t)n_sub;
            int64_t p = 0, k = sub_base[c], sub_start = 0;
            for (int64_t i = chunk_start[c]; i < chunk_end[c] && rc == CO3O_OK; i++) {
                uint32_t cw = 0;
                int found = -1;
                for (int l2 = 1; l2 <= CO3O_MAXLEN && found < 0; l2++) {
                    if (p >= avail) { rc = CO3O_ECORRUPT; break; }
                    cw = (cw << 1) | (uint32_t)get_bit(words, p++);
                    if (cn[l2] && cw >= fi[l2] && cw - fi[l2] < cn[l2]) found = so[st[l2] + (cw - fi[l2])];
                }
                if (found < 0) { rc = CO3O_ECORRUPT; break; }
                int64_t kk = co3o_K(E, M, found & ((1 << nm) - 1));
                ksum[i - chunk_start[c]] += (found >> nm) ? -kk : kk;
                if (sym_out) sym_out[(size_t)u * (size_t)sld + i] = (uint8_t)found;
                if ((i + 1) % CO3O_SUB == 0 || i + 1 == chunk_end[c]) {
                    if (p - sub_start != (int64_t)sb[k]) { rc = CO3O_ECORRUPT; break; }
                    sub_start = p; k++;
                }
            }
        }
        if (rc != CO3O_OK) break;
        float scale = (float)ldexp(1.0, hdr[3 * l + 0] + co3o_cF(E, M));
        for (int64_t i = 0; i < n; i++) {
            volatile float prod = (float)ksum[i] * scale;       /* exact */
            volatile float a = prod / (float)U;
            avg[chunk_start[c] + i] = a;
        }
    }
    free(ksum); free(len); free(code); free(w); free(first); free(count); free(start); free(sorted);
    return rc;
}
