// Fused user-side pass of Algorithm 1 lines 8 and 10 (sm_100a):
//   a = g + gamma m;  ghat = Q_fp(a);  m <- a - ghat
// plus what the code design needs from the same data: the symbol histogram per segment and the
// moments sum|a|, sum a^2 of a (the GenNorm model is fitted to g_t + gamma m_{t-1}).
//
// Bound: HBM.  Per user-element 8 B read (g, m), 4 B (m) + 1 B (symbol) written.  All global
// accesses are 128-bit (4 B for the packed symbols) on a 4096-element tile grid that is aligned
// in the row, so segment boundaries never misalign the vectors; the vectors that straddle a
// chunk edge are handled element by element.
//
// Work item = (user, chunk).  Blocks are persistent and take contiguous item ranges, so a block
// stays inside one segment for long stretches: the histogram lives in shared memory (one copy
// per warp) and is flushed with 64-bit global atomics only when the segment changes.  Moments
// are reduced in a fixed order per item and stored per item, so the fit does not depend on the
// launch geometry or on scheduling.
#include "co3_internal.h"

namespace {

struct QParams {
    int lambda;        // grid value = K * 2^lambda
    float inv_scale;   // 2^-lambda
    float top;         // K_max * 2^lambda
    int M, nm;
};

__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

// Q_fp on one element.  Round-to-nearest-even at the quantum of a's binade (or the subnormal
// quantum 2^lambda, whichever is larger) by adding and subtracting 1.5 * 2^(qe+23); saturate;
// then read the magnitude code off the bits of the integer magnitude.
template <bool CONVERT>
__device__ __forceinline__ void ef_element(float g, float m, float gamma, const QParams& q,
                                           uint32_t& sym, float& m_new, double& s1, double& s2,
                                           uint32_t& nf) {
    const float a = __fadd_rn(g, __fmul_rn(gamma, m));
    const uint32_t ab = __float_as_uint(a);
    if (((ab >> 23) & 0xFFu) == 0xFFu) {      // NaN / Inf: counted, coded as +0, memory reset
        nf += 1;
        sym = 0;
        m_new = 0.0f;
        return;
    }
    const float ax = fabsf(a);
    const double ad = (double)ax;
    s1 += ad;
    s2 = __fma_rn(ad, ad, s2);                // ad*ad is exact in double, so this rounds once
    if (!CONVERT) return;
    const float axc = fminf(ax, q.top);
    const int pa = (int)(__float_as_uint(axc) >> 23) - 127;
    const int qe = max(pa - q.M, q.lambda);
    const float magic = __uint_as_float(((uint32_t)(qe + 23 + 127) << 23) | 0x400000u);
    const float r = __fsub_rn(__fadd_rn(axc, magic), magic);   // multiple of 2^qe, <= top
    const float kf = __fmul_rn(r, q.inv_scale);                 // integer magnitude, exact
    const uint32_t k = (uint32_t)kf;
    const uint32_t kb = __float_as_uint(kf);
    const uint32_t j = (k < (2u << q.M)) ? k
                                         : ((kb >> (23 - q.M)) - ((uint32_t)(127 + q.M - 1) << q.M));
    const uint32_t s = (ab >> 31) & (uint32_t)(k != 0);
    sym = (s << q.nm) | j;
    m_new = __fsub_rn(a, s ? -r : r);
}

template <bool CONVERT>
__global__ void __launch_bounds__(CO3_THREADS)
ef_kernel(Co3Dev p, const float* __restrict__ g, float* __restrict__ m) {
    __shared__ uint32_t s_hist[CO3_THREADS / 32][CO3_MAXSYM];
    __shared__ double s_red[2][2][CO3_THREADS / 32];
    __shared__ uint32_t s_rednf[2][CO3_THREADS / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t n_items = p.n_chunks * (int64_t)p.U;
    const int64_t per = (n_items + gridDim.x - 1) / gridDim.x;
    const int64_t it0 = (int64_t)blockIdx.x * per;
    const int64_t it1 = min(n_items, it0 + per);
    if (it0 >= it1) return;

    if (CONVERT) {
        for (int i = tid; i < (CO3_THREADS / 32) * CO3_MAXSYM; i += CO3_THREADS) (&s_hist[0][0])[i] = 0;
        __syncthreads();
    }
    int cur_seg = -1;
    QParams q;
    q.M = p.M; q.nm = p.nm; q.lambda = 0; q.inv_scale = 1.0f; q.top = 0.0f;

    for (int64_t item = it0; item < it1; ++item) {
        const int u = (int)(item / p.n_chunks);
        const int64_t c = item - (int64_t)u * p.n_chunks;
        const Co3Chunk cd = p.chunks[c];
        if (CONVERT && cd.seg != cur_seg) {
            if (cur_seg >= 0) {               // flush the histogram of the segment just left
                __syncthreads();
                if (tid < p.nsym) {
                    unsigned long long tot = 0;
#pragma unroll
                    for (int w = 0; w < CO3_THREADS / 32; ++w) { tot += s_hist[w][tid]; s_hist[w][tid] = 0; }
                    if (tot) atomicAdd(&p.hist[(size_t)cur_seg * CO3_MAXSYM + tid], tot);
                }
                __syncthreads();
            }
            cur_seg = cd.seg;
            q.lambda = p.bias_cur[cd.seg] + p.cF;
            q.inv_scale = pow2f(-q.lambda);
            q.top = __fmul_rn((float)p.Kmax, pow2f(q.lambda));
        }
        const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
        const int lo = (int)(cd.start - tb), hi = lo + cd.len;
        const float* gr = g + (size_t)u * p.ld + tb;
        float* mr = m + (size_t)u * p.ld + tb;
        uint8_t* sr = p.sym + (size_t)u * p.sld + tb;

        float4 gv[4], mv[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int e0 = 4 * (tid + CO3_THREADS * r);
            if (e0 < hi && e0 + 4 > lo) {
                gv[r] = __ldg(reinterpret_cast<const float4*>(gr + e0));
                mv[r] = *reinterpret_cast<const float4*>(mr + e0);
            }
        }
        double s1 = 0.0, s2 = 0.0;
        uint32_t nf = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int e0 = 4 * (tid + CO3_THREADS * r);
            if (!(e0 < hi && e0 + 4 > lo)) continue;
            const float ge[4] = {gv[r].x, gv[r].y, gv[r].z, gv[r].w};
            const float me[4] = {mv[r].x, mv[r].y, mv[r].z, mv[r].w};
            float mo[4];
            uint32_t so[4];
            const bool full = (e0 >= lo) && (e0 + 4 <= hi);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                so[e] = 0; mo[e] = 0.0f;
                if (full || (e0 + e >= lo && e0 + e < hi)) {
                    ef_element<CONVERT>(ge[e], me[e], p.gamma, q, so[e], mo[e], s1, s2, nf);
                    if (CONVERT) atomicAdd(&s_hist[warp][so[e]], 1u);
                }
            }
            if (CONVERT) {
                if (full) {
                    *reinterpret_cast<float4*>(mr + e0) = make_float4(mo[0], mo[1], mo[2], mo[3]);
                    *reinterpret_cast<uint32_t*>(sr + e0) = so[0] | (so[1] << 8) | (so[2] << 16) | (so[3] << 24);
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (e0 + e >= lo && e0 + e < hi) { mr[e0 + e] = mo[e]; sr[e0 + e] = (uint8_t)so[e]; }
                }
            }
        }
        // fixed-order reduction of this item's moments: lanes, then warps
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s1 += __shfl_down_sync(0xffffffffu, s1, o);
            s2 += __shfl_down_sync(0xffffffffu, s2, o);
            nf += __shfl_down_sync(0xffffffffu, nf, o);
        }
        const int par = (int)(item & 1);
        if (lane == 0) { s_red[par][0][warp] = s1; s_red[par][1][warp] = s2; s_rednf[par][warp] = nf; }
        __syncthreads();
        if (tid == 0) {
            double t1 = 0.0, t2 = 0.0;
            uint32_t tn = 0;
#pragma unroll
            for (int w = 0; w < CO3_THREADS / 32; ++w) { t1 += s_red[par][0][w]; t2 += s_red[par][1][w]; tn += s_rednf[par][w]; }
            p.part_s1[item] = t1; p.part_s2[item] = t2; p.part_nf[item] = tn;
        }
    }
    if (CONVERT && cur_seg >= 0) {
        __syncthreads();
        if (tid < p.nsym) {
            unsigned long long tot = 0;
#pragma unroll
            for (int w = 0; w < CO3_THREADS / 32; ++w) tot += s_hist[w][tid];
            if (tot) atomicAdd(&p.hist[(size_t)cur_seg * CO3_MAXSYM + tid], tot);
        }
    }
}

int g_ef_blocks_per_sm[2] = {0, 0};

}  // namespace

static int ef_grid(const co3_plan* pl, int which) {
    if (g_ef_blocks_per_sm[which] == 0) {
        int n = 0;
        if (which) cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, ef_kernel<true>, CO3_THREADS, 0);
        else cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, ef_kernel<false>, CO3_THREADS, 0);
        g_ef_blocks_per_sm[which] = n > 0 ? n : 1;
    }
    int64_t items = pl->dev.n_chunks * (int64_t)pl->dev.U;
    int64_t grid = (int64_t)pl->num_sms * g_ef_blocks_per_sm[which];
    return (int)(items < grid ? items : grid);
}

cudaError_t co3_launch_stats(co3_plan* pl, const float* g, const float* m, cudaStream_t st) {
    co3_prof_begin(pl, CO3_K_STATS, st);
    ef_kernel<false><<<ef_grid(pl, 0), CO3_THREADS, 0, st>>>(pl->dev, g, const_cast<float*>(m));
    co3_prof_end(pl, CO3_K_STATS, st, 1);
    return cudaGetLastError();
}

cudaError_t co3_launch_convert(co3_plan* pl, const float* g, float* m, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(pl->dev.hist, 0, sizeof(unsigned long long) * (size_t)pl->dev.S * CO3_MAXSYM, st);
    if (e != cudaSuccess) return e;
    co3_prof_begin(pl, CO3_K_CONVERT, st);
    ef_kernel<true><<<ef_grid(pl, 1), CO3_THREADS, 0, st>>>(pl->dev, g, m);
    co3_prof_end(pl, CO3_K_CONVERT, st, 1);
    return cudaGetLastError();
}
