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
// launch geometry or on scheduling.  A thread handles one 4-element vector per step (4 steps per
// item) and always has the next step's two 128-bit loads in flight (register double buffer that
// runs across item boundaries), so with four resident blocks per SM the memory system stays full
// while the conversion arithmetic runs.
#include "co3_internal.h"

namespace {

constexpr int STEPS = CO3_TILE / (4 * CO3_THREADS);   // vectors per thread per item (4)

struct QParams {
    int lambda;        // grid value = K * 2^lambda
    float inv_scale;   // 2^-lambda
    float top;         // K_max * 2^lambda
};

__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

// Q_fp on one element.  Round-to-nearest-even at the quantum of a's binade (or the subnormal
// quantum 2^lambda, whichever is larger) by adding and subtracting 1.5 * 2^(qe+23); saturate;
// then read the magnitude code off the bits of the integer magnitude.  M = mantissa bits,
// NM = exponent + mantissa bits (position of the sign in the symbol byte).
template <int M, bool CONVERT>
__device__ __forceinline__ void ef_element(float g, float m, float gamma, const QParams& q, int nm,
                                           uint32_t& sym, float& m_new, double& s1, double& s2,
                                           uint32_t& nf) {
    const float a = __fadd_rn(g, __fmul_rn(gamma, m));
    const uint32_t ab = __float_as_uint(a);
    if ((ab & 0x7F800000u) == 0x7F800000u) {  // NaN / Inf: counted, coded as +0, memory reset
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
    const int qe = max((int)(__float_as_uint(axc) >> 23) - (127 + M), q.lambda);
    const float magic = __uint_as_float((uint32_t)(qe << 23) + ((150u << 23) | 0x400000u));
    const float r = __fsub_rn(__fadd_rn(axc, magic), magic);   // multiple of 2^qe, <= top
    const float kf = __fmul_rn(r, q.inv_scale);                 // integer magnitude, exact
    const uint32_t k = (uint32_t)kf;
    const uint32_t j = (k < (2u << M)) ? k : ((__float_as_uint(kf) >> (23 - M)) - ((uint32_t)(127 + M - 1) << M));
    const uint32_t s = (k != 0) ? (ab >> 31) : 0u;
    sym = (s << nm) | j;
    m_new = __fsub_rn(a, __uint_as_float(__float_as_uint(r) | (s << 31)));
}

struct ItemCtx {                  // what a step needs to know about its item
    const float* gr;              // row pointers at the start of the item's tile
    float* mr;
    uint8_t* sr;
    int lo, hi;                   // the item's elements within the tile
};

template <int M, bool CONVERT>
__global__ void __launch_bounds__(CO3_THREADS, CONVERT ? 4 : 4)
ef_kernel(Co3Dev p, const float* __restrict__ g, float* __restrict__ m) {
    __shared__ uint32_t s_hist[CONVERT ? CO3_THREADS / 32 : 1][CO3_MAXSYM];
    __shared__ double s_red[2][2][CO3_THREADS / 32];
    __shared__ uint32_t s_rednf[2][CO3_THREADS / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_items = (uint32_t)p.n_chunks * (uint32_t)p.U;
    const uint32_t per = (n_items + gridDim.x - 1) / gridDim.x;
    const uint32_t it0 = blockIdx.x * per;
    const uint32_t it1 = min(n_items, it0 + per);
    if (it0 >= it1) return;

    if (CONVERT) {
        for (int i = tid; i < (CO3_THREADS / 32) * CO3_MAXSYM; i += CO3_THREADS) (&s_hist[0][0])[i] = 0;
        __syncthreads();
    }
    const int nm = p.nm;
    const uint32_t n_chunks = (uint32_t)p.n_chunks;
    uint32_t u = it0 / n_chunks, c = it0 - u * n_chunks;

    auto make_ctx = [&](uint32_t uu, const Co3Chunk& cd) {
        ItemCtx x;
        const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
        x.gr = g + (size_t)uu * p.ld + tb;
        x.mr = m + (size_t)uu * p.ld + tb;
        x.sr = p.sym + (size_t)uu * p.sld + tb;
        x.lo = (int)(cd.start - tb);
        x.hi = x.lo + cd.len;
        return x;
    };
    auto load_step = [&](const ItemCtx& x, int r, float4& gv, float4& mv) {
        const int e0 = 4 * (tid + CO3_THREADS * r);
        if (e0 < x.hi && e0 + 4 > x.lo) {
            gv = __ldg(reinterpret_cast<const float4*>(x.gr + e0));
            mv = *reinterpret_cast<const float4*>(x.mr + e0);
        }
    };

    Co3Chunk cd = p.chunks[c];
    ItemCtx cur = make_ctx(u, cd);
    float4 gbuf[2], mbuf[2];
    load_step(cur, 0, gbuf[0], mbuf[0]);

    int cur_seg = -1;
    QParams q;
    q.lambda = 0; q.inv_scale = 1.0f; q.top = 0.0f;

    for (uint32_t item = it0; item < it1; ++item) {
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
        // the next item (for the prefetch that crosses the item boundary)
        uint32_t un = u, cn = c + 1;
        if (cn == n_chunks) { cn = 0; ++un; }
        const bool has_next = item + 1 < it1;
        Co3Chunk cdn = cd;
        ItemCtx nxt = cur;
        if (has_next) { cdn = p.chunks[cn]; nxt = make_ctx(un, cdn); }

        double s1 = 0.0, s2 = 0.0;
        uint32_t nf = 0;
#pragma unroll
        for (int r = 0; r < STEPS; ++r) {
            // keep the next step's loads in flight while this one is converted
            if (r + 1 < STEPS) load_step(cur, r + 1, gbuf[(r + 1) & 1], mbuf[(r + 1) & 1]);
            else if (has_next) load_step(nxt, 0, gbuf[0], mbuf[0]);
            const int e0 = 4 * (tid + CO3_THREADS * r);
            if (!(e0 < cur.hi && e0 + 4 > cur.lo)) continue;
            const float4 gv = gbuf[r & 1], mv = mbuf[r & 1];
            const float ge[4] = {gv.x, gv.y, gv.z, gv.w};
            const float me[4] = {mv.x, mv.y, mv.z, mv.w};
            float mo[4];
            uint32_t so[4];
            const bool full = (e0 >= cur.lo) && (e0 + 4 <= cur.hi);
            if (full) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    ef_element<M, CONVERT>(ge[e], me[e], p.gamma, q, nm, so[e], mo[e], s1, s2, nf);
                    if (CONVERT) atomicAdd(&s_hist[warp][so[e]], 1u);
                }
                if (CONVERT) {
                    *reinterpret_cast<float4*>(cur.mr + e0) = make_float4(mo[0], mo[1], mo[2], mo[3]);
                    *reinterpret_cast<uint32_t*>(cur.sr + e0) = so[0] | (so[1] << 8) | (so[2] << 16) | (so[3] << 24);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (e0 + e >= cur.lo && e0 + e < cur.hi) {
                        ef_element<M, CONVERT>(ge[e], me[e], p.gamma, q, nm, so[e], mo[e], s1, s2, nf);
                        if (CONVERT) {
                            atomicAdd(&s_hist[warp][so[e]], 1u);
                            cur.mr[e0 + e] = mo[e];
                            cur.sr[e0 + e] = (uint8_t)so[e];
                        }
                    }
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
        u = un; c = cn; cd = cdn; cur = nxt;
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

typedef void (*ef_fn)(Co3Dev, const float*, float*);

template <bool CONVERT>
ef_fn pick_kernel(int M) {
    switch (M) {
        case 1: return ef_kernel<1, CONVERT>;
        case 2: return ef_kernel<2, CONVERT>;
        case 3: return ef_kernel<3, CONVERT>;
        case 4: return ef_kernel<4, CONVERT>;
        case 5: return ef_kernel<5, CONVERT>;
        default: return ef_kernel<6, CONVERT>;
    }
}

int ef_grid(const co3_plan* pl, ef_fn fn) {
    int n = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, CO3_THREADS, 0);
    if (n < 1) n = 1;
    const int64_t items = pl->dev.n_chunks * (int64_t)pl->dev.U;
    const int64_t grid = (int64_t)pl->num_sms * n;
    return (int)(items < grid ? items : grid);
}

}  // namespace

cudaError_t co3_launch_stats(co3_plan* pl, const float* g, const float* m, cudaStream_t st) {
    ef_fn fn = pick_kernel<false>(pl->dev.M);
    if (!pl->grid_stats) pl->grid_stats = ef_grid(pl, fn);
    co3_prof_begin(pl, CO3_K_STATS, st);
    fn<<<pl->grid_stats, CO3_THREADS, 0, st>>>(pl->dev, g, const_cast<float*>(m));
    co3_prof_end(pl, CO3_K_STATS, st, 1);
    return cudaGetLastError();
}

cudaError_t co3_launch_convert(co3_plan* pl, const float* g, float* m, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(pl->dev.hist, 0, sizeof(unsigned long long) * (size_t)pl->dev.S * CO3_MAXSYM, st);
    if (e != cudaSuccess) return e;
    ef_fn fn = pick_kernel<true>(pl->dev.M);
    if (!pl->grid_convert) pl->grid_convert = ef_grid(pl, fn);
    co3_prof_begin(pl, CO3_K_CONVERT, st);
    fn<<<pl->grid_convert, CO3_THREADS, 0, st>>>(pl->dev, g, m);
    co3_prof_end(pl, CO3_K_CONVERT, st, 1);
    return cudaGetLastError();
}
