// Small per-segment / per-model-row kernels (sm_100a):
//  * fit_kernel      -- pooled moments -> GenNorm shape/scale by moment matching -> exponent bias
//                       (Eq. "approximate") and the header indices that name the code model.
//                       Runs once per iteration (twice when the bias is taken from the current
//                       iteration's own moments).
//  * huff_cand_kernel / code_finalize_kernel -- element-wise Huffman code of the quantised GenNorm
//                       model (Sec. III (ii)), canonical codewords, encoder and decoder tables,
//                       for EVERY model row.  A code depends only on the format and on the two
//                       header indices, so these run once, when the plan is created; an iteration
//                       only selects rows.
// All are latency-bound.  The moment ratio is inverted through a table of log R(beta) (uniform in
// log2 beta) by a two-level parallel search and inverse cubic interpolation, so the solve costs no
// lgamma evaluation; the depth limit of the code is resolved by building every weight-floor
// candidate in its own block.
#include "co3_internal.h"
#include "co3_quant.cuh"

namespace {

constexpr int FIT_THREADS = 512;   // reduction width
constexpr int FIT_SEARCH = 128;    // = FIT_GRID / 64: one coarse table interval per searching thread
constexpr long long FIT_REDO_MAX = 8192;   // user-elements of a layer that the fit's own block converts again (mode 6)

__device__ __forceinline__ double poly_bias(double b) {
    const double b2 = b * b;
    return 0.46 - 2.85 * b + 5.37 * b2 - 2.85 * b2 * b + 0.52 * b2 * b2;
}

// Plans with very long segments (millions of (user, chunk) pairs): slice blockIdx.x of segment
// blockIdx.y adds its contiguous share of the pairs, in a fixed order, so that the fit kernel has
// only red_k numbers per segment left to add.
constexpr int RED_THREADS = 256;
__global__ void __launch_bounds__(RED_THREADS) fit_reduce_kernel(Co3Dev p, int clear_enc_sync) {
    __shared__ double s_a[RED_THREADS / 32], s_b[RED_THREADS / 32];
    __shared__ unsigned long long s_n[RED_THREADS / 32];
    const int seg = blockIdx.x, slice = blockIdx.y, tid = threadIdx.x;   // (the x extent has no 65535 limit)
    if (clear_enc_sync) {                              // (see fit_kernel: here the many blocks share that job)
        const size_t nb = (size_t)gridDim.x * gridDim.y, b = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
        for (size_t i = b * RED_THREADS + tid; i < p.enc_sync_words64; i += nb * RED_THREADS) p.enc_grp[i] = 0ull;
    }
    const int c0 = p.seg_chunk0[seg], nck = p.seg_chunk0[seg + 1] - c0;
    const long long npairs = (long long)nck * p.U;
    const long long per = (npairs + p.red_k - 1) / p.red_k;
    const long long lo = per * slice, hi = min(npairs, lo + per);
    double a1 = 0.0, a2 = 0.0;
    unsigned long long an = 0;
#pragma unroll 4
    for (long long k = lo + tid; k < hi; k += RED_THREADS) {
        const long long u = k / nck;
        const size_t i = (size_t)u * (size_t)p.n_chunks + c0 + (size_t)(k - u * nck);
        a1 += p.part_s1[i];
        a2 += p.part_s2[i];
        an += p.part_nf[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a1 += __shfl_down_sync(0xffffffffu, a1, o);
        a2 += __shfl_down_sync(0xffffffffu, a2, o);
        an += __shfl_down_sync(0xffffffffu, an, o);
    }
    if ((tid & 31) == 0) { s_a[tid >> 5] = a1; s_b[tid >> 5] = a2; s_n[tid >> 5] = an; }
    __syncthreads();
    if (tid == 0) {
        double t1 = 0.0, t2 = 0.0;
        unsigned long long tn = 0;
#pragma unroll
        for (int w = 0; w < RED_THREADS / 32; ++w) { t1 += s_a[w]; t2 += s_b[w]; tn += s_n[w]; }
        const size_t o = (size_t)seg * p.red_k + slice;
        p.red_s1[o] = t1; p.red_s2[o] = t2; p.red_nf[o] = tn;
    }
}

// mode 0: after the stats pass -- write the bias for the coming convert pass.
// mode 1: after the convert pass -- write the header (bias used, ibeta, ir), keep the fit, and
//         store the bias the rule gives for these moments as the next iteration's bias.
// Fully lagged code (the whole header of an iteration is fixed before its gradient is seen):
// mode 2: after the stats pass of t = 0 -- bias and header of the coming pass from these moments.
// mode 3: after the fused convert-and-pack pass -- the same for the next iteration; keep the fit.
//         In both, `hdr` is the plan's own header array.
// mode 4: only add up the moments of every segment and write (N, S1, S2) to mom_out.
// mode 5: after the stats pass when the bias comes from the current iteration's own moments: the bias for
//         the coming convert pass AND the header of this iteration (the convert pass sums the same
//         a = g + gamma m item by item in the same order, so a second fit after it would reproduce these
//         numbers bit for bit); keeps the fit and prepares the encoder like mode 1.
// mode 6: after a convert pass that ran under a GUESSED bias (bias_cur, the previous iteration's) although the
//         bias is to come from this iteration's own moments: bias and header from these moments as in mode 5;
//         a layer whose bias differs from the guess is put on the list of layers to convert again,
//         and bias_cur takes the bias found (the re-conversion's target and
//         the next iteration's guess).
// ext_mom (may be null): (N, S1, S2) per segment that replace the plan's own sums in the fit (the sums
//         of a layer that is spread over several plans); the non-finite count stays the plan's own.
// fit_ovr (may be null): (beta, alpha) per segment that replace the solve (test hook: a harness feeds
//         another implementation's fit to tell a rounding of the fit from a fault further down).
// clear_hist: the convert pass is the next launch; its histogram and item ticket are zeroed here
//         (a memset of its own between the two kernels costs the step two microseconds).
__global__ void __launch_bounds__(FIT_THREADS) fit_kernel(Co3Dev p, int mode, co3_seg_header* hdr,
                                                          const double* __restrict__ ext_mom,
                                                          double* __restrict__ mom_out,
                                                          const double* __restrict__ fit_ovr, int clear_hist,
                                                          float* __restrict__ residual) {
    __shared__ double s_a[FIT_THREADS / 32], s_b[FIT_THREADS / 32];
    __shared__ unsigned long long s_n[FIT_THREADS / 32];
    __shared__ double s_lg[3];
    __shared__ double s_target, s_t;        // log rho; log2(beta)
    __shared__ int s_state, s_coarse, s_fine;
    __shared__ double s_ct[FIT_SEARCH + 1];  // log R at every 64th grid point (the coarse level of the search)
    __shared__ double s_fx[68], s_fg[68];   // log R and log G around the bracket: grid points i0 - 1 .. i0 + 66
    __shared__ int s_redo_old;              // mode 6: the guess this layer was converted with, if this block converts it again
    __shared__ uint32_t s_rh[2][CO3_MAXSYM];

    const int seg = blockIdx.x, tid = threadIdx.x;
    if ((mode == 1 || mode == 5 || mode == 6) && p.red_k == 0) {
        // side job: the single-pass encode that follows this launch wants its tickets, published
        // counts and group totals at zero
        unsigned long long* z = p.enc_grp;
        for (size_t i = (size_t)blockIdx.x * FIT_THREADS + tid; i < p.enc_sync_words64; i += (size_t)gridDim.x * FIT_THREADS) z[i] = 0ull;
    }
    if (clear_hist) {
        for (int h = 0; h < p.hist_copies; ++h)
            for (int i = tid; i < CO3_MAXSYM; i += FIT_THREADS) p.hist[((size_t)h * p.S + seg) * CO3_MAXSYM + i] = 0ull;
        if (seg == 0 && tid == 0) *p.ticket = 0u;
    }
    const int c0 = p.seg_chunk0[seg], c1 = p.seg_chunk0[seg + 1];
    // fixed order: thread t takes the (user, chunk) pairs t, t + 512, ... of the segment, all loads
    // independent; then lanes, then warps.  (Plans with very long segments: the pairs were summed in
    // red_k slices by fit_reduce_kernel, and the slices are added here.)
    const int nck = c1 - c0, npairs = nck * p.U;
    // the coarse level of the search table: on its way while the partial sums are added up
    if (tid <= FIT_SEARCH && mode != 4) s_ct[tid] = p.logr_tab[tid * (CO3_FIT_GRID / FIT_SEARCH)];
    if (mode == 6 && tid < 2 && nck > 0)              // should this block convert its layer again: descriptor and side-list count on their way
        asm volatile("prefetch.global.L2 [%0];" ::"l"(tid == 0 ? (const void*)(p.chunks + c0) : (const void*)(p.spec + 2)));
    double a1 = 0.0, a2 = 0.0;
    unsigned long long an = 0;
    if (p.red_k > 0) {
        for (int k = tid; k < p.red_k; k += FIT_THREADS) {
            const size_t i = (size_t)seg * p.red_k + k;
            a1 += p.red_s1[i];
            a2 += p.red_s2[i];
            an += p.red_nf[i];
        }
    } else {
#pragma unroll 4
        for (int k = tid; k < npairs; k += FIT_THREADS) {
            const int u = k / nck, c = c0 + (k - u * nck);
            const size_t i = (size_t)u * (size_t)p.n_chunks + c;
            a1 += p.part_s1[i];
            a2 += p.part_s2[i];
            an += p.part_nf[i];
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a1 += __shfl_down_sync(0xffffffffu, a1, o);
        a2 += __shfl_down_sync(0xffffffffu, a2, o);
        an += __shfl_down_sync(0xffffffffu, an, o);
    }
    if ((tid & 31) == 0) { s_a[tid >> 5] = a1; s_b[tid >> 5] = a2; s_n[tid >> 5] = an; }
    __syncthreads();
    double S1 = 0.0, S2 = 0.0;
    unsigned long long nf = 0;
#pragma unroll
    for (int w = 0; w < FIT_THREADS / 32; ++w) { S1 += s_a[w]; S2 += s_b[w]; nf += s_n[w]; }
    double N = (double)((unsigned long long)(p.seg_off[seg + 1] - p.seg_off[seg]) * (unsigned long long)p.U - nf);
    if (mode == 4) {
        if (tid == 0) { mom_out[3 * seg] = N; mom_out[3 * seg + 1] = S1; mom_out[3 * seg + 2] = S2; }
        return;
    }
    if (ext_mom) { N = ext_mom[3 * seg]; S1 = ext_mom[3 * seg + 1]; S2 = ext_mom[3 * seg + 2]; }

    // beta = clamp(R^-1(rho), 0.3, 2.0), rho = N S2 / S1^2; R is strictly decreasing in beta, and
    // the tables hold log R and log G at log2(beta) = T0 + i * H.
    const double T0 = log2(0.3), H = (1.0 - T0) / (double)CO3_FIT_GRID;
    const double* tab = p.logr_tab;
    const double* tabg = p.logr_tab + CO3_FIT_GRID + 1;
    if (tid < 3) s_lg[tid] = log(tid == 0 ? N : (tid == 1 ? S2 : S1));   // three logarithms side by side
    __syncthreads();
    if (tid == 0) {
        s_state = 0; s_coarse = 0; s_fine = 0;
        if (fit_ovr) { s_state = fit_ovr[2 * seg + 1] > 0.0 ? 3 : 2; s_t = 0.0; }   // given; alpha = 0: as below
        else if (!(N > 0.0) || !(S1 > 0.0)) { s_state = 2; s_t = 0.0; }     // beta = 1, alpha = 0
        else {
            s_target = s_lg[0] + s_lg[1] - 2.0 * s_lg[2];
            if (s_target >= s_ct[0]) { s_state = 1; s_t = T0; s_fine = 0; }
            else if (s_target <= s_ct[FIT_SEARCH]) { s_state = 1; s_t = 1.0; s_fine = CO3_FIT_GRID; }
        }
    }
    __syncthreads();
    if (s_state == 0) {
        // interval i with tab[i] > target >= tab[i+1]: coarse then fine, 64 entries each
        constexpr int STEP = CO3_FIT_GRID / FIT_SEARCH;        // 64
        const double target = s_target;
        if (tid < FIT_SEARCH && s_ct[tid] > target && target >= s_ct[tid + 1]) s_coarse = tid;
        __syncthreads();
        // one round of loads brings the bracket's 64 intervals and the nodes of both interpolations
        const int i0 = s_coarse * STEP;
        if (tid < 68) {
            const int gi = min(max(i0 - 1 + tid, 0), CO3_FIT_GRID);
            s_fx[tid] = tab[gi];
            s_fg[tid] = tabg[gi];
        }
        __syncthreads();
        if (tid < STEP && s_fx[tid + 1] > target && target >= s_fx[tid + 2]) s_fine = i0 + tid;
        __syncthreads();
    }
    constexpr int NO_REDO = -(1 << 30);
    if (tid == 0) s_redo_old = NO_REDO;
    if (tid == 0) [&]() {                   // the solve, by one thread
    double t = s_t, beta, log_g;
    if (s_state == 0) {
        // inverse cubic (Lagrange) interpolation of log2(beta) as a function of log R through the
        // four grid points around the bracket, then cubic interpolation of log G at that point
        int i = s_fine;
        i = i < 1 ? 1 : (i > CO3_FIT_GRID - 2 ? CO3_FIT_GRID - 2 : i);
        const double target = s_target;
        double xs[4], gs[4], acc = 0.0;
        const int o = i - (s_coarse * (CO3_FIT_GRID / FIT_SEARCH));      // 0 .. 63 within the bracket (clamped at the table's ends)
        for (int k = 0; k < 4; ++k) { xs[k] = s_fx[o + k]; gs[k] = s_fg[o + k]; }
        for (int a = 0; a < 4; ++a) {
            double term = T0 + H * (double)(i - 1 + a);
            for (int c = 0; c < 4; ++c)
                if (c != a) term *= (target - xs[c]) / (xs[a] - xs[c]);
            acc += term;
        }
        t = acc;
        const double x = (t - (T0 + H * (double)(i - 1))) / H;           // position among the four nodes 0..3
        log_g = gs[0] * ((x - 1.0) * (x - 2.0) * (x - 3.0) / -6.0) + gs[1] * (x * (x - 2.0) * (x - 3.0) / 2.0) +
                gs[2] * (x * (x - 1.0) * (x - 3.0) / -2.0) + gs[3] * (x * (x - 1.0) * (x - 2.0) / 6.0);
        beta = exp2(t);
    } else if (s_state == 1) {
        beta = (t == T0) ? 0.3 : 2.0;
        log_g = tabg[s_fine];
    } else if (s_state == 3) {
        beta = fit_ovr[2 * seg];
        log_g = 0.0;
    } else {
        beta = 1.0;
        log_g = 0.0;
    }
    const double log2e = 1.4426950408889634;
    // alpha = (S1 / N) * G(beta); its base-2 logarithm without forming alpha first
    const double log2_alpha = (s_state == 2) ? 0.0 : (s_state == 3 ? log2(fit_ovr[2 * seg + 1]) : (s_lg[2] - s_lg[0] + log_g) * log2e);
    const bool has_alpha = s_state != 2;
    const double alpha = has_alpha ? (s_state == 3 ? fit_ovr[2 * seg + 1] : exp2(log2_alpha)) : 0.0;
    int b_rule = p.b_lo;
    if (has_alpha && alpha > 0.0) {
        if (p.bias_rule == CO3_RULE_OPT) {
            // the integer bias of least expected squared error: (round(8 log2 alpha) - best ir) / 8
            double xb = floor(8.0 * (s_state == 0 ? t : log2(beta)) + 0.5);
            xb = xb < (double)CO3_IBETA_MIN ? (double)CO3_IBETA_MIN : (xb > (double)CO3_IBETA_MAX ? (double)CO3_IBETA_MAX : xb);
            const double t8 = floor(8.0 * log2_alpha + 0.5);
            if (t8 < -16000.0) b_rule = p.b_lo;
            else if (t8 > 16000.0) b_rule = p.b_hi;
            else {
                const int ti = (int)t8, rho = ((ti % 8) + 8) % 8;
                const int b = (ti - (int)p.bias_opt_tab[((int)xb - CO3_IBETA_MIN) * 8 + rho]) / 8;   // exact
                b_rule = b < p.b_lo ? p.b_lo : (b > p.b_hi ? p.b_hi : b);
            }
        } else {
            const double bf = floor(log2_alpha - log2(poly_bias(beta)) + 0.5);
            b_rule = bf < (double)p.b_lo ? p.b_lo : (bf > (double)p.b_hi ? p.b_hi : (int)bf);
        }
    }
    if (mode == 0) {
        p.bias_cur[seg] = b_rule;
        return;
    }
    const int b_used = (mode == 1) ? p.bias_cur[seg] : b_rule;   // the bias this header goes with
    double x = floor(8.0 * (s_state == 0 ? t : log2(beta)) + 0.5);
    x = x < (double)CO3_IBETA_MIN ? (double)CO3_IBETA_MIN : (x > (double)CO3_IBETA_MAX ? (double)CO3_IBETA_MAX : x);
    double y = (double)CO3_IR_MIN;
    if (has_alpha && alpha > 0.0) {
        y = floor(8.0 * (log2_alpha - (double)b_used) + 0.5);
        y = y < (double)CO3_IR_MIN ? (double)CO3_IR_MIN : (y > (double)CO3_IR_MAX ? (double)CO3_IR_MAX : y);
    }
    co3_seg_header h;
    h.bias = (int8_t)b_used; h.ibeta = (int8_t)(int)x; h.ir = (int16_t)(int)y;
    hdr[seg] = h;
    // (a layer of zeros converts to the same symbols and memory under every bias: nothing to repair)
    if (mode == 6 && b_rule != p.bias_cur[seg] && S1 > 0.0) {
        // a small layer is converted again by this very block (below); a large one by the pass that follows
        if ((long long)(p.seg_off[seg + 1] - p.seg_off[seg]) * p.U <= FIT_REDO_MAX) s_redo_old = p.bias_cur[seg];
        else {
            const int k = atomicAdd(p.spec, 1);
            p.redo_seg[k] = seg;
            p.redo_old[k] = p.bias_cur[seg];
        }
    }
    // Bias from the current moments: bias_cur is the next conversion's GUESS (and, for a layer that is
    // converted again, the bias to convert it to).  After a layer of zeros the rule's bias is the lowest one,
    // under which the first non-zero gradient would saturate beyond recovery; the highest one turns
    // everything into zeros with the element itself as memory, from which any bias can be reached.
    p.bias_cur[seg] = ((mode == 5 || mode == 6) && !(S1 > 0.0)) ? p.b_hi : b_rule;
    if (mode == 2) return;
    double* f = p.fit + 5 * (size_t)seg;
    f[0] = beta; f[1] = alpha; f[2] = N; f[3] = S1; f[4] = S2;
    if (nf) {
        atomicAdd(p.nonfinite_total, nf);
        atomicOr(p.flags, CO3_FLAG_NONFINITE);
    }
    }();
    if (mode != 6) return;
    __syncthreads();
    if (s_redo_old == NO_REDO) return;
    // mode 6, a small layer whose bias differs from the guess: converted again here (the layers that keep
    // the convert pass busy for microseconds go on the list instead, for all SMs to share)
    const int b_new = p.bias_cur[seg];      // (written by thread 0 before the barrier)
    switch (p.M) {
        case 1: redo_small<1>(p, residual, seg, c0, nck, s_redo_old, b_new, tid, FIT_THREADS, s_rh); redo_side_of_layer<1>(p, residual, seg, tid, FIT_THREADS); break;
        case 2: redo_small<2>(p, residual, seg, c0, nck, s_redo_old, b_new, tid, FIT_THREADS, s_rh); redo_side_of_layer<2>(p, residual, seg, tid, FIT_THREADS); break;
        case 3: redo_small<3>(p, residual, seg, c0, nck, s_redo_old, b_new, tid, FIT_THREADS, s_rh); redo_side_of_layer<3>(p, residual, seg, tid, FIT_THREADS); break;
        case 4: redo_small<4>(p, residual, seg, c0, nck, s_redo_old, b_new, tid, FIT_THREADS, s_rh); redo_side_of_layer<4>(p, residual, seg, tid, FIT_THREADS); break;
        case 5: redo_small<5>(p, residual, seg, c0, nck, s_redo_old, b_new, tid, FIT_THREADS, s_rh); redo_side_of_layer<5>(p, residual, seg, tid, FIT_THREADS); break;
        default: redo_small<6>(p, residual, seg, c0, nck, s_redo_old, b_new, tid, FIT_THREADS, s_rh); redo_side_of_layer<6>(p, residual, seg, tid, FIT_THREADS); break;
    }
}

// One (model row, weight floor 2^cand) pair per block: Huffman code lengths of the floored model
// weights.  Leaves sorted by (weight, symbol); two queues; on equal weights the leaf goes first.
// FROM_HIST: the row is a segment and the weights are this iteration's symbol counts (all copies of
// the histogram added, low bits dropped until the segment's total is below 2^31).
template <bool FROM_HIST>
__global__ void __launch_bounds__(CO3_MAXSYM) huff_cand_kernel(Co3Dev p, Co3CodeBook cb) {
    typedef unsigned long long W;                    // floors go up to 2^31: node weights need 64 bits
    constexpr W NONE = ~(W)0;
    __shared__ W s_w[CO3_MAXSYM], s_sw[CO3_MAXSYM], s_iw[CO3_MAXSYM];
    __shared__ uint16_t s_ssym[CO3_MAXSYM], s_parent[2 * CO3_MAXSYM];
    __shared__ int s_max;
    const int rowi = blockIdx.x, cand = blockIdx.y, tid = threadIdx.x, n = p.nsym;
    if (tid == 0) s_max = 0;
    if (tid < n) {
        uint32_t w;
        if (FROM_HIST) {
            const unsigned long long tot = (unsigned long long)(p.seg_off[rowi + 1] - p.seg_off[rowi]) * (unsigned long long)p.U;
            int k = 0;
            while ((tot >> k) >= (1ull << 31)) ++k;
            unsigned long long c = 0;
            for (int h = 0; h < p.hist_copies; ++h)
                c += p.hist[((size_t)h * p.S + rowi) * CO3_MAXSYM + co3_sym_internal(tid, p.nm)];
            w = (uint32_t)(c >> k);
        } else {
            const int j = tid & (p.J - 1);
            w = ((tid >> p.nm) && j == 0) ? 1u : p.wtab[(size_t)rowi * p.J + j];   // "-0" is never emitted
        }
        s_w[tid] = max((W)w, (W)1 << cand);
    }
    __syncthreads();
    if (tid < n) {
        const W mine = s_w[tid];
        int rank = 0;
        for (int s = 0; s < n; ++s) {
            const W o = s_w[s];
            rank += (o < mine) || (o == mine && s < tid);
        }
        s_sw[rank] = mine;
        s_ssym[rank] = (uint16_t)tid;
    }
    __syncthreads();
    if (tid == 0) {
        int i = 0, j = 0;
        W lw = s_sw[0];                              // head of the leaf queue
        W iw = NONE;                                 // head of the internal queue (none yet)
        for (int k = 0; k < n - 1; ++k) {
            W sum = 0;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (lw <= iw) {                      // leaf first on ties; NONE when exhausted
                    sum += lw;
                    s_parent[i] = (uint16_t)(n + k);
                    ++i;
                    lw = (i < n) ? s_sw[i] : NONE;
                } else {
                    sum += iw;
                    s_parent[n + j] = (uint16_t)(n + k);
                    ++j;
                    iw = (j < k) ? s_iw[j] : NONE;
                }
            }
            s_iw[k] = sum;
            if (j == k) iw = sum;                    // the node just made becomes the queue head
        }
    }
    __syncthreads();
    if (tid < n) {
        const int root = 2 * n - 2;
        int node = tid, depth = 0;
        while (node != root && depth <= CO3_MAXLEN) { node = s_parent[node]; ++depth; }
        atomicMax(&s_max, depth);
        cb.cand_len[((size_t)rowi * cb.ncand + cand) * CO3_MAXSYM + s_ssym[tid]] = (uint8_t)depth;
    }
    __syncthreads();
    if (tid == 0) cb.cand_max[rowi * cb.ncand + cand] = s_max;
}

// Per model row: take the smallest floor whose code is at most 16 deep, assign canonical
// codewords (symbols ordered by (length, symbol)), and write the encoder table and the decoder
// tables (13-bit primary table, second table for the codewords of 12 bits and more, canonical arrays).
// FROM_LENS: the lengths are given (lens_in, [rows][2^B] by public symbol: the side information of the
// empirical-histogram code on the decoding side); lengths that are not those of a complete prefix
// code raise CO3_FLAG_CORRUPT.  lens_out (may be null): the chosen lengths, same layout.
template <bool FROM_LENS>
__global__ void __launch_bounds__(CO3_MAXSYM) code_finalize_kernel(Co3Dev p, Co3CodeBook cb,
                                                                   const uint8_t* __restrict__ lens_in,
                                                                   uint8_t* __restrict__ lens_out) {
    __shared__ uint8_t s_len[CO3_MAXSYM], s_perm[CO3_MAXSYM];
    __shared__ uint32_t s_count[CO3_MAXLEN + 2], s_first[CO3_MAXLEN + 2], s_offs[CO3_MAXLEN + 2];
    __shared__ int s_sel;
    const int rowi = blockIdx.x, tid = threadIdx.x, n = p.nsym;
    if (tid == 0 && !FROM_LENS) {
        int sel = cb.ncand - 1;                          // the last floor always passes (see CO3_NCAND*)
        for (int c = 0; c < cb.ncand; ++c)
            if (cb.cand_max[rowi * cb.ncand + c] <= CO3_MAXLEN) { sel = c; break; }
        s_sel = sel;
    }
    if (tid < CO3_MAXLEN + 2) s_count[tid] = 0;
    __syncthreads();
    if (tid < n) {
        uint8_t L;
        if (FROM_LENS) {
            L = lens_in[(size_t)rowi * n + tid];
            if (L < 1 || L > CO3_MAXLEN) { L = CO3_MAXLEN; atomicOr(p.flags, CO3_FLAG_CORRUPT); }
        } else {
            L = cb.cand_len[((size_t)rowi * cb.ncand + s_sel) * CO3_MAXSYM + tid];
            if (L > CO3_MAXLEN) L = CO3_MAXLEN;            // cannot happen: the last floor passes
            if (lens_out) lens_out[(size_t)rowi * n + tid] = L;
        }
        s_len[tid] = L;
        atomicAdd(&s_count[L], 1u);
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t code = 0, off = 0, kraft = 0;
        for (int L = 1; L <= CO3_MAXLEN; ++L) {
            s_first[L] = code; s_offs[L] = off;
            code = (code + s_count[L]) << 1;
            off += s_count[L];
            kraft += s_count[L] << (CO3_MAXLEN - L);
        }
        if (FROM_LENS && kraft != (1u << CO3_MAXLEN)) atomicOr(p.flags, CO3_FLAG_CORRUPT);
    }
    __syncthreads();
    if (tid < n) {
        const int L = s_len[tid];
        uint32_t r = 0;
        for (int s = 0; s < tid; ++s) r += (s_len[s] == L);
        const uint32_t code = s_first[L] + r;
        const uint32_t rev = __brev(code) >> (32 - L);
        const size_t o = (size_t)rowi * CO3_MAXSYM + tid;
        const size_t oi = (size_t)rowi * CO3_MAXSYM + co3_sym_internal(tid, p.nm);
        cb.len8[oi] = (uint8_t)L;                   // the encoder looks up stored (internal) symbols
        cb.enc[oi] = rev | ((uint32_t)L << 16);
        cb.len_pub[o] = (uint8_t)L;
        cb.code_msb[o] = code;
        s_perm[s_offs[L] + r] = (uint8_t)tid;
        if (rowi == 0) cb.ksign[tid] = co3_ksigned(tid, p.M, p.nm);
    }
    __syncthreads();
    if (tid < n) cb.perm[(size_t)rowi * CO3_MAXSYM + tid] = s_perm[tid];
    if (tid <= CO3_MAXLEN) {
        const size_t o = (size_t)rowi * (CO3_MAXLEN + 1) + tid;
        cb.first[o] = tid ? s_first[tid] : 0;
        cb.count[o] = tid ? s_count[tid] : 0;
        cb.offs[o] = tid ? s_offs[tid] : 0;
    }
    for (int i = tid; i < CO3_LUT_SIZE; i += CO3_MAXSYM) {
        const uint32_t v = __brev((uint32_t)i) >> (32 - CO3_LUT_BITS);   // stream order -> root bit on top
        uint32_t entry = 0;
        for (int L = 1; L <= CO3_LUT_BITS; ++L) {
            const uint32_t dd = (v >> (CO3_LUT_BITS - L)) - s_first[L];
            if (dd < s_count[L]) {
                const int sym = s_perm[s_offs[L] + dd];
                entry = ((uint32_t)co3_ksigned(sym, p.M, p.nm) << 8) | (uint32_t)L;
                break;
            }
        }
        cb.lut[(size_t)rowi * CO3_LUT_SIZE + i] = entry;
    }
    // Second table for the codewords a primary table of 11 or 13 bits cannot hold.  Canonical codes grow with the length,
    // so every 16-bit window that starts with a codeword of 12..16 bits is >= first[12] << 4, and
    // there are at most 16 per symbol of them.
    const uint32_t long_first = s_first[CO3_LONG_FROM] << (CO3_MAXLEN - CO3_LONG_FROM);
    for (int i = tid; i < cb.long_stride; i += CO3_MAXSYM) {
        const uint32_t v = long_first + (uint32_t)i;          // 16 stream bits, root bit on top
        uint32_t entry = 0;                                    // 0: no codeword starts like this
        if (v < (1u << CO3_MAXLEN)) {
            for (int L = CO3_LONG_FROM; L <= CO3_MAXLEN; ++L) {
                const uint32_t dd = (v >> (CO3_MAXLEN - L)) - s_first[L];
                if (dd < s_count[L]) {
                    const int sym = s_perm[s_offs[L] + dd];
                    entry = ((uint32_t)co3_ksigned(sym, p.M, p.nm) << 8) | (uint32_t)L;
                    break;
                }
            }
        }
        cb.lut_long[(size_t)rowi * cb.long_stride + i] = entry;
    }
}

}  // namespace

cudaError_t co3_launch_fit(co3_plan* pl, int mode, co3_seg_header* hdr, cudaStream_t st, bool clear_hist, float* residual) {
    co3_prof_begin(pl, CO3_K_FIT, st);
    if (pl->dev.red_k > 0) fit_reduce_kernel<<<dim3(pl->dev.S, pl->dev.red_k), RED_THREADS, 0, st>>>(pl->dev, mode == 1 || mode == 5 || mode == 6);
    const double* ext = (pl->use_ext_mom && mode != 4) ? pl->ext_mom : nullptr;
    if (mode != 4) pl->use_ext_mom = false;                // imported moments serve one fit
    fit_kernel<<<pl->dev.S, FIT_THREADS, 0, st>>>(pl->dev, mode, hdr, ext, pl->mom_out,
                                                  (pl->use_fit_ovr && mode != 4) ? pl->fit_ovr : nullptr, clear_hist ? 1 : 0, residual);
    co3_prof_end(pl, CO3_K_FIT, st, pl->dev.red_k > 0 ? 2 : 1);
    return cudaGetLastError();
}

// Builds the code tables of all model rows (plan creation).
cudaError_t co3_build_codebook(co3_plan* pl, cudaStream_t st) {
    dim3 grid(CO3_NROWS, CO3_NCAND);
    huff_cand_kernel<false><<<grid, CO3_MAXSYM, 0, st>>>(pl->dev, pl->dev.cb);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    code_finalize_kernel<false><<<CO3_NROWS, CO3_MAXSYM, 0, st>>>(pl->dev, pl->dev.cb, nullptr, nullptr);
    return cudaGetLastError();
}

// Empirical-histogram code, encoding side: one Huffman code per segment from the histogram the
// convert pass has just filled; the lengths go to code_lens as well (the side information).
cudaError_t co3_build_hist_codes(co3_plan* pl, uint8_t* code_lens, cudaStream_t st) {
    dim3 grid(pl->dev.S, CO3_NCAND_HIST);
    co3_prof_begin(pl, CO3_K_CODE_ENC, st);
    huff_cand_kernel<true><<<grid, CO3_MAXSYM, 0, st>>>(pl->dev, pl->cb_emp);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) {
        code_finalize_kernel<false><<<pl->dev.S, CO3_MAXSYM, 0, st>>>(pl->dev, pl->cb_emp, nullptr, code_lens);
        e = cudaGetLastError();
    }
    co3_prof_end(pl, CO3_K_CODE_ENC, st, 2);
    return e;
}

// Empirical-histogram code, decoding side: the tables of the canonical codes with the given lengths.
cudaError_t co3_build_codes_from_lens(co3_plan* pl, const uint8_t* code_lens, cudaStream_t st) {
    co3_prof_begin(pl, CO3_K_CODE_DEC, st);
    code_finalize_kernel<true><<<pl->dev.S, CO3_MAXSYM, 0, st>>>(pl->dev, pl->cb_emp, code_lens, nullptr);
    co3_prof_end(pl, CO3_K_CODE_DEC, st, 1);
    return cudaGetLastError();
}
