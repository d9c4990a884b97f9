// Small per-segment kernels between the streaming passes (sm_100a):
//  * fit_kernel      -- pooled moments -> GenNorm shape/scale by moment matching -> exponent bias
//                       (Eq. "approximate") and the header indices that name the code model.
//  * huff_cand_kernel / code_finalize_kernel -- element-wise Huffman code of the quantised GenNorm
//                       model (Sec. III (ii)), canonical codewords, encoder and decoder tables.
// All are latency-bound (O(segments * alphabet) work); they are organised so that the serial part
// of each (one two-queue merge of <= 255 steps) runs once, with every weight-floor candidate of
// the depth limit in its own block.
#include "co3_internal.h"

namespace {

constexpr int FIT_THREADS = 128;
constexpr int FIT_POINTS = 42;   // interior points per search round (3 lgamma each = 126 threads)
constexpr int FIT_ROUNDS = 9;    // (hi - lo) shrinks by 43 per round: 1.7 / 43^9 < 4e-15

__device__ __forceinline__ double poly_bias(double b) {
    const double b2 = b * b;
    return 0.46 - 2.85 * b + 5.37 * b2 - 2.85 * b2 * b + 0.52 * b2 * b2;
}

// log R(beta) = lgamma(1/b) + lgamma(3/b) - 2 lgamma(2/b) at K points, three threads per point.
__device__ void eval_logR(const double* pts, int K, double* out, double* s_lg, int tid) {
    if (tid < 3 * K) s_lg[tid] = lgamma((double)(tid % 3 + 1) / pts[tid / 3]);
    __syncthreads();
    if (tid < K) out[tid] = s_lg[3 * tid] + s_lg[3 * tid + 2] - 2.0 * s_lg[3 * tid + 1];
    __syncthreads();
}

// mode 0: after the stats pass -- write the bias for the coming convert pass.
// mode 1: after the convert pass -- write the header (bias used, ibeta, ir), keep the fit, and
//         store the bias the rule gives for these moments as the next iteration's bias.
__global__ void __launch_bounds__(FIT_THREADS) fit_kernel(Co3Dev p, int mode, co3_seg_header* hdr) {
    __shared__ double s_a[FIT_THREADS], s_b[FIT_THREADS];
    __shared__ unsigned long long s_n[FIT_THREADS];
    __shared__ double s_pts[FIT_POINTS + 2], s_val[FIT_POINTS + 2], s_lg[3 * (FIT_POINTS + 2)];
    __shared__ double s_lo, s_hi, s_target;
    __shared__ int s_state;   // 0 search, 1 beta fixed in s_lo

    const int seg = blockIdx.x, tid = threadIdx.x;
    const int c0 = p.seg_chunk0[seg], c1 = p.seg_chunk0[seg + 1];
    const int64_t nci = c1 - c0, total = nci * p.U;
    double a1 = 0.0, a2 = 0.0;
    unsigned long long an = 0;
    for (int64_t k = tid; k < total; k += FIT_THREADS) {
        const int64_t u = k / nci, c = c0 + (k - u * nci);
        const int64_t idx = u * p.n_chunks + c;
        a1 += p.part_s1[idx];
        a2 += p.part_s2[idx];
        an += p.part_nf[idx];
    }
    s_a[tid] = a1; s_b[tid] = a2; s_n[tid] = an;
    __syncthreads();
    for (int o = FIT_THREADS / 2; o > 0; o >>= 1) {
        if (tid < o) { s_a[tid] += s_a[tid + o]; s_b[tid] += s_b[tid + o]; s_n[tid] += s_n[tid + o]; }
        __syncthreads();
    }
    const double S1 = s_a[0], S2 = s_b[0];
    const unsigned long long nf = s_n[0];
    const double N = (double)((unsigned long long)(p.seg_off[seg + 1] - p.seg_off[seg]) * (unsigned long long)p.U - nf);
    __syncthreads();

    // beta = clamp(R^-1(rho), 0.3, 2.0), rho = N S2 / S1^2, R strictly decreasing
    if (tid == 0) {
        s_state = 0;
        if (!(N > 0.0) || !(S1 > 0.0)) { s_state = 2; s_lo = 1.0; }
        else s_target = log(N) + log(S2) - 2.0 * log(S1);
        s_pts[0] = 0.3; s_pts[1] = 2.0;
    }
    __syncthreads();
    if (s_state == 0) {
        eval_logR(s_pts, 2, s_val, s_lg, tid);
        if (tid == 0) {
            if (s_target >= s_val[0]) { s_state = 1; s_lo = 0.3; }
            else if (s_target <= s_val[1]) { s_state = 1; s_lo = 2.0; }
            else { s_lo = 0.3; s_hi = 2.0; }
        }
        __syncthreads();
    }
    if (s_state == 0) {
        for (int round = 0; round < FIT_ROUNDS; ++round) {
            if (tid < FIT_POINTS) s_pts[tid] = s_lo + (s_hi - s_lo) * ((double)(tid + 1) / (double)(FIT_POINTS + 1));
            __syncthreads();
            eval_logR(s_pts, FIT_POINTS, s_val, s_lg, tid);
            if (tid == 0) {
                double lo = s_lo, hi = s_hi;
                for (int k = 0; k < FIT_POINTS; ++k) {
                    if (s_val[k] > s_target) lo = s_pts[k];
                    else { hi = s_pts[k]; break; }
                }
                s_lo = lo; s_hi = hi;
            }
            __syncthreads();
        }
        if (tid == 0) s_lo = 0.5 * (s_lo + s_hi);
        __syncthreads();
    }
    const double beta = s_lo;
    if (tid < 2) s_lg[tid] = lgamma((double)(tid + 1) / beta);
    __syncthreads();
    if (tid != 0) return;

    const double alpha = (s_state == 2) ? 0.0 : (S1 / N) * exp(s_lg[0] - s_lg[1]);
    int b_rule = p.b_lo;
    if (alpha > 0.0) {
        const double bf = floor(log2(alpha) - log2(poly_bias(beta)) + 0.5);
        b_rule = bf < (double)p.b_lo ? p.b_lo : (bf > (double)p.b_hi ? p.b_hi : (int)bf);
    }
    if (mode == 0) {
        p.bias_cur[seg] = b_rule;
        return;
    }
    const int b_used = p.bias_cur[seg];
    double x = floor(8.0 * log2(beta) + 0.5);
    x = x < (double)CO3_IBETA_MIN ? (double)CO3_IBETA_MIN : (x > (double)CO3_IBETA_MAX ? (double)CO3_IBETA_MAX : x);
    double y = (double)CO3_IR_MIN;
    if (alpha > 0.0) {
        y = floor(8.0 * (log2(alpha) - (double)b_used) + 0.5);
        y = y < (double)CO3_IR_MIN ? (double)CO3_IR_MIN : (y > (double)CO3_IR_MAX ? (double)CO3_IR_MAX : y);
    }
    co3_seg_header h;
    h.bias = (int8_t)b_used; h.ibeta = (int8_t)(int)x; h.ir = (int16_t)(int)y;
    hdr[seg] = h;
    double* f = p.fit + 5 * (size_t)seg;
    f[0] = beta; f[1] = alpha; f[2] = N; f[3] = S1; f[4] = S2;
    p.bias_cur[seg] = b_rule;
    if (nf) {
        atomicAdd(p.nonfinite_total, nf);
        atomicOr(p.flags, CO3_FLAG_NONFINITE);
    }
}

// One (segment, weight floor 2^cand) pair per block: Huffman code lengths of the floored model
// weights.  Leaves sorted by (weight, symbol); two queues; on equal weights the leaf goes first.
__global__ void __launch_bounds__(CO3_MAXSYM)
huff_cand_kernel(Co3Dev p, Co3CodeBook cb, const co3_seg_header* __restrict__ hdr) {
    __shared__ uint32_t s_w[CO3_MAXSYM], s_sw[CO3_MAXSYM], s_iw[CO3_MAXSYM];
    __shared__ uint16_t s_ssym[CO3_MAXSYM], s_parent[2 * CO3_MAXSYM];
    __shared__ int s_max;
    const int seg = blockIdx.x, cand = blockIdx.y, tid = threadIdx.x, n = p.nsym;
    const co3_seg_header h = hdr[seg];
    int ib = (int)h.ibeta, ir = (int)h.ir;
    if (ib < CO3_IBETA_MIN || ib > CO3_IBETA_MAX || ir < CO3_IR_MIN || ir > CO3_IR_MAX) {
        if (tid == 0 && cand == 0) atomicOr(p.flags, CO3_FLAG_CORRUPT);   // header out of range
        ib = min(max(ib, CO3_IBETA_MIN), CO3_IBETA_MAX);
        ir = min(max(ir, CO3_IR_MIN), CO3_IR_MAX);
    }
    const uint32_t* row = p.wtab + ((size_t)(ib - CO3_IBETA_MIN) * CO3_NIR + (ir - CO3_IR_MIN)) * p.J;
    if (tid == 0) s_max = 0;
    if (tid < n) {
        const int j = tid & (p.J - 1);
        const uint32_t w = ((tid >> p.nm) && j == 0) ? 1u : row[j];
        s_w[tid] = max(w, 1u << cand);
    }
    __syncthreads();
    if (tid < n) {
        const uint32_t mine = s_w[tid];
        int rank = 0;
        for (int s = 0; s < n; ++s) {
            const uint32_t o = s_w[s];
            rank += (o < mine) || (o == mine && s < tid);
        }
        s_sw[rank] = mine;
        s_ssym[rank] = (uint16_t)tid;
    }
    __syncthreads();
    if (tid == 0) {
        int i = 0, j = 0;
        uint32_t lw = s_sw[0];                       // head of the leaf queue
        uint32_t iw = 0xFFFFFFFFu;                   // head of the internal queue (none yet)
        for (int k = 0; k < n - 1; ++k) {
            uint32_t sum = 0;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (lw <= iw) {                      // leaf first on ties; lw = UINT_MAX when exhausted
                    sum += lw;
                    s_parent[i] = (uint16_t)(n + k);
                    ++i;
                    lw = (i < n) ? s_sw[i] : 0xFFFFFFFFu;
                } else {
                    sum += iw;
                    s_parent[n + j] = (uint16_t)(n + k);
                    ++j;
                    iw = (j < k) ? s_iw[j] : 0xFFFFFFFFu;
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
        cb.cand_len[((size_t)seg * CO3_NCAND + cand) * CO3_MAXSYM + s_ssym[tid]] = (uint8_t)depth;
    }
    __syncthreads();
    if (tid == 0) cb.cand_max[seg * CO3_NCAND + cand] = s_max;
}

// Per segment: take the smallest floor whose code is at most 16 deep, assign canonical
// codewords (symbols ordered by (length, symbol)), and write the encoder table and, if asked,
// the decoder tables (11-bit primary table + canonical arrays for the rare longer codewords).
__global__ void __launch_bounds__(CO3_MAXSYM)
code_finalize_kernel(Co3Dev p, Co3CodeBook cb, int want_decode) {
    __shared__ uint8_t s_len[CO3_MAXSYM], s_perm[CO3_MAXSYM];
    __shared__ uint32_t s_count[CO3_MAXLEN + 2], s_first[CO3_MAXLEN + 2], s_offs[CO3_MAXLEN + 2];
    __shared__ int s_sel;
    const int seg = blockIdx.x, tid = threadIdx.x, n = p.nsym;
    if (tid == 0) {
        int sel = CO3_NCAND - 1;
        for (int c = 0; c < CO3_NCAND; ++c)
            if (cb.cand_max[seg * CO3_NCAND + c] <= CO3_MAXLEN) { sel = c; break; }
        s_sel = sel;
    }
    if (tid < CO3_MAXLEN + 2) s_count[tid] = 0;
    __syncthreads();
    if (tid < n) {
        const uint8_t L = cb.cand_len[((size_t)seg * CO3_NCAND + s_sel) * CO3_MAXSYM + tid];
        s_len[tid] = L;
        atomicAdd(&s_count[L], 1u);
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t code = 0, off = 0;
        for (int L = 1; L <= CO3_MAXLEN; ++L) {
            s_first[L] = code; s_offs[L] = off;
            code = (code + s_count[L]) << 1;
            off += s_count[L];
        }
    }
    __syncthreads();
    if (tid < n) {
        const int L = s_len[tid];
        uint32_t r = 0;
        for (int s = 0; s < tid; ++s) r += (s_len[s] == L);
        const uint32_t code = s_first[L] + r;
        const uint32_t rev = __brev(code) >> (32 - L);
        const size_t o = (size_t)seg * CO3_MAXSYM + tid;
        cb.len8[o] = (uint8_t)L;
        cb.enc[o] = rev | ((uint32_t)L << 16);
        cb.code_msb[o] = code;
        s_perm[s_offs[L] + r] = (uint8_t)tid;
        if (want_decode) cb.ksign[o] = co3_ksigned(tid, p.M, p.nm);
    }
    __syncthreads();
    if (!want_decode) return;
    if (tid < n) cb.perm[(size_t)seg * CO3_MAXSYM + tid] = s_perm[tid];
    if (tid <= CO3_MAXLEN) {
        const size_t o = (size_t)seg * (CO3_MAXLEN + 1) + tid;
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
        cb.lut[(size_t)seg * CO3_LUT_SIZE + i] = entry;
    }
}

}  // namespace

cudaError_t co3_launch_fit(co3_plan* pl, int mode, co3_seg_header* hdr, cudaStream_t st) {
    co3_prof_begin(pl, CO3_K_FIT, st);
    fit_kernel<<<pl->dev.S, FIT_THREADS, 0, st>>>(pl->dev, mode, hdr);
    co3_prof_end(pl, CO3_K_FIT, st, 1);
    return cudaGetLastError();
}

cudaError_t co3_launch_codebook(co3_plan* pl, const Co3CodeBook& cb, const co3_seg_header* hdr,
                                int want_decode_tables, cudaStream_t st) {
    const int k = want_decode_tables ? CO3_K_CODE_DEC : CO3_K_CODE_ENC;
    dim3 grid(pl->dev.S, CO3_NCAND);
    co3_prof_begin(pl, k, st);
    huff_cand_kernel<<<grid, CO3_MAXSYM, 0, st>>>(pl->dev, cb, hdr);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) {
        code_finalize_kernel<<<pl->dev.S, CO3_MAXSYM, 0, st>>>(pl->dev, cb, want_decode_tables);
        e = cudaGetLastError();
    }
    co3_prof_end(pl, k, st, 2);
    return e;
}
