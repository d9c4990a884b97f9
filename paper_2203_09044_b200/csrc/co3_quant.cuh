// The quantiser Q_fp of Algorithm 1 line 10 and the re-conversion of a layer under another bias, for
// the kernels that need them (the convert pass, the re-conversion pass, the fit).  Device code only.
#pragma once
#include "co3_internal.h"

struct QParams {                 // per segment
    float top;                   // K_max * 2^lambda: largest grid value (grid value = K * 2^lambda)
    uint32_t low_bits;           // bits of 2^(lambda + M): below it the quantum stays 2^lambda
    uint32_t e0;                 // exponent field of 1.5 * 2^(lambda + 23): lambda + 150
    uint32_t far_bits;           // conversion under a guessed bias: bits of 2^(23 - M) * top (capped at those of Inf)
};

__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

template <int M>
__device__ __forceinline__ QParams make_qparams(uint32_t Kmax, int lambda) {
    QParams q;
    q.top = __fmul_rn((float)Kmax, pow2f(lambda));
    q.low_bits = __float_as_uint(pow2f(lambda + M));
    q.e0 = (uint32_t)(lambda + 150);
    q.far_bits = min(__float_as_uint(q.top) + ((23u - M) << 23), 0x7F800000u);   // top < 2^100: stays below the sign bit
    return q;
}

// Q_fp on one finite element, branch-free.  |a| (clamped to the top grid value) is rounded to
// nearest even at the quantum 2^qe of its binade -- or the subnormal quantum 2^lambda, whichever
// is larger -- by adding 1.5 * 2^(qe+23): the sum t holds n = |a| / 2^qe rounded, as an integer, in
// its low mantissa bits, and subtracting the constant again gives the rounded value r.  The
// magnitude code is j = ((qe - lambda) << M) + n for every binade (n < 2^(M+1) below the second
// binade, where it is the code itself; 2^M <= n <= 2^(M+1) above, where it carries the mantissa
// and, on a carry, the next exponent).
template <int M>
__device__ __forceinline__ void quantize(float a, const QParams& q, uint32_t& sym, float& m_new) {
    const uint32_t ab = __float_as_uint(a);
    const float axc = fminf(fabsf(a), q.top);
    // exponent field of max(|a|, 2^(lambda+M)), moved up by 23 - M binades, plus the 1.5
    const uint32_t mb = (max(__float_as_uint(axc), q.low_bits) & 0x7F800000u) + (((23u - M) << 23) | 0x400000u);
    const float magic = __uint_as_float(mb);
    const float t = __fadd_rn(axc, magic);
    const float r = __fsub_rn(t, magic);      // multiple of 2^qe, <= top
    const uint32_t tb = __float_as_uint(t);
    const uint32_t j = (((tb >> 23) - q.e0) << M) + (tb & 0x3FFFFFu);
    const uint32_t sb = (r != 0.0f) ? (ab & 0x80000000u) : 0u;  // "-0" is never emitted
    sym = (j << 1) | (sb >> 31);                                 // internal form: code << 1 | sign
    m_new = __fsub_rn(a, __uint_as_float(__float_as_uint(r) | sb));
}

// a from its grid value and its new memory (exact for every element that is not on the side list; qv = 0
// leaves a itself, sign of zero included).
__device__ __forceinline__ float rebuild_a(float qv, float m_new) { return qv == 0.0f ? m_new : __fadd_rn(qv, m_new); }

// One vector of four elements (e0 .. e0 + 3 of the tile whose rows start at mrow / srow) of a layer that
// was converted at the bias behind quantum_old: every a = q + m' is rebuilt from the stored symbol and
// memory and converted again with q; s_hist[0] counts the symbols taken out, s_hist[1] those put in.
template <int M>
__device__ __forceinline__ void redo_vector(float* mrow, uint8_t* srow, int e0, int lo, int hi, const QParams& q,
                                            float quantum_old, uint32_t (*s_hist)[CO3_MAXSYM]) {
    if (e0 >= hi || e0 + 4 <= lo) return;
    if (e0 >= lo && e0 + 4 <= hi) {
        const uint32_t sw = *reinterpret_cast<const uint32_t*>(srow + e0);
        const float4 mv = *reinterpret_cast<const float4*>(mrow + e0);
        const float mold[4] = {mv.x, mv.y, mv.z, mv.w};
        uint32_t so[4];
        float mo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t sy = (sw >> (8 * e)) & 0xFFu;
            const float qv = __fmul_rn((float)co3_ksigned_internal((int)sy, M), quantum_old);   // exact
            quantize<M>(rebuild_a(qv, mold[e]), q, so[e], mo[e]);
            atomicAdd(&s_hist[0][sy], 1u);
            atomicAdd(&s_hist[1][so[e]], 1u);
        }
        *reinterpret_cast<float4*>(mrow + e0) = make_float4(mo[0], mo[1], mo[2], mo[3]);
        *reinterpret_cast<uint32_t*>(srow + e0) = so[0] | (so[1] << 8) | (so[2] << 16) | (so[3] << 24);
    } else {                                          // a vector on the chunk's edge: element by element
        for (int e = 0; e < 4; ++e) {
            if (e0 + e < lo || e0 + e >= hi) continue;
            const uint32_t sy = srow[e0 + e];
            const float qv = __fmul_rn((float)co3_ksigned_internal((int)sy, M), quantum_old);
            uint32_t so;
            float mo;
            quantize<M>(rebuild_a(qv, mrow[e0 + e]), q, so, mo);
            atomicAdd(&s_hist[0][sy], 1u);
            atomicAdd(&s_hist[1][so], 1u);
            mrow[e0 + e] = mo;
            srow[e0 + e] = (uint8_t)so;
        }
    }
}

// The difference of the two counts goes to the layer's histogram (into copy 0: the copies are summed when
// the histogram is read).
__device__ __forceinline__ void redo_flush(const Co3Dev& p, int seg, int tid, int nthreads, uint32_t (*s_hist)[CO3_MAXSYM]) {
    __syncthreads();
    for (int i = tid; i < CO3_MAXSYM; i += nthreads)
        if (s_hist[0][i] != s_hist[1][i])
            atomicAdd(&p.hist[(size_t)seg * CO3_MAXSYM + i], (unsigned long long)s_hist[1][i] - (unsigned long long)s_hist[0][i]);
    __syncthreads();
}

// A layer (chunks c0 .. c0 + nck - 1 of every user) converted again, bias b_old -> b_new.  Items (user, chunk)
// it0, it0 + it_step, ... are this block's, a thread takes the vectors tid, tid + nthreads, ... of a tile;
// called by all threads of the block.
template <int M>
__device__ void redo_items(const Co3Dev& p, float* __restrict__ m, int seg, int c0, int nck, int b_old, int b_new,
                           int64_t it0, int64_t it_step, int tid, int nthreads, uint32_t (*s_hist)[CO3_MAXSYM]) {
    const QParams q = make_qparams<M>(p.Kmax, b_new + p.cF);
    const float quantum_old = pow2f(b_old + p.cF);
    const int64_t n_it = (int64_t)nck * p.U;
    for (int i = tid; i < 2 * CO3_MAXSYM; i += nthreads) (&s_hist[0][0])[i] = 0;
    __syncthreads();
    for (int64_t it = it0; it < n_it; it += it_step) {
        const int u = (int)(it / nck);
        const Co3Chunk cd = p.chunks[c0 + (int)(it - (int64_t)u * nck)];
        const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
        const int lo = (int)(cd.start - tb), hi = lo + cd.len;
        for (int e0 = 4 * tid; e0 < CO3_TILE; e0 += 4 * nthreads)
            redo_vector<M>(m + (size_t)u * p.ld + tb, p.sym + (size_t)u * p.sld + tb, e0, lo, hi, q, quantum_old, s_hist);
    }
    redo_flush(p, seg, tid, nthreads, s_hist);
}

// The same for a small layer, by one block: the vectors of all users of a chunk side by side, so that a
// layer of a few hundred elements is one round of loads.
template <int M>
__device__ void redo_small(const Co3Dev& p, float* __restrict__ m, int seg, int c0, int nck, int b_old, int b_new,
                           int tid, int nthreads, uint32_t (*s_hist)[CO3_MAXSYM]) {
    const QParams q = make_qparams<M>(p.Kmax, b_new + p.cF);
    const float quantum_old = pow2f(b_old + p.cF);
    for (int i = tid; i < 2 * CO3_MAXSYM; i += nthreads) (&s_hist[0][0])[i] = 0;
    __syncthreads();
    for (int ci = 0; ci < nck; ++ci) {
        const Co3Chunk cd = p.chunks[c0 + ci];
        const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
        const int lo = (int)(cd.start - tb), hi = lo + cd.len;
        const int v_lo = lo >> 2, nv = ((hi + 3) >> 2) - v_lo;
        for (int f = tid; f < nv * p.U; f += nthreads) {
            const int u = f / nv, e0 = 4 * (v_lo + (f - u * nv));
            redo_vector<M>(m + (size_t)u * p.ld + tb, p.sym + (size_t)u * p.sld + tb, e0, lo, hi, q, quantum_old, s_hist);
        }
    }
    redo_flush(p, seg, tid, nthreads, s_hist);
}

// An element of the side list whose layer has been converted again: the value the convert pass kept is
// converted in place of the rebuilt one, and the histogram follows.
template <int M>
__device__ __forceinline__ void redo_side_entry(const Co3Dev& p, float* __restrict__ m, const Co3Side& e, const Co3Chunk& cd,
                                                uint32_t user) {
    const int64_t i = (cd.start & ~(int64_t)(CO3_TILE - 1)) + e.pos;       // element index in the user's row
    const QParams q = make_qparams<M>(p.Kmax, p.bias_cur[cd.seg] + p.cF);
    uint32_t so;
    float mo;
    quantize<M>(__uint_as_float(e.a_bits), q, so, mo);
    uint8_t* sp = p.sym + (size_t)user * p.sld + i;
    atomicAdd(&p.hist[(size_t)cd.seg * CO3_MAXSYM + *sp], ~0ull);          // minus one: the symbol that the rebuilt value gave
    atomicAdd(&p.hist[(size_t)cd.seg * CO3_MAXSYM + so], 1ull);
    *sp = (uint8_t)so;
    m[(size_t)user * p.ld + i] = mo;
}

// The side-list entries of layer `seg`, after that layer has been converted again by this block.
template <int M>
__device__ void redo_side_of_layer(const Co3Dev& p, float* __restrict__ m, int seg, int tid, int nthreads) {
    const int n_side = min(p.spec[2], CO3_SIDE_CAP);
    for (int j = tid; j < n_side; j += nthreads) {
        const Co3Side e = p.side[j];
        const uint32_t user = e.item / (uint32_t)p.n_chunks;
        const Co3Chunk cd = p.chunks[e.item - user * (uint32_t)p.n_chunks];
        if (cd.seg == seg) redo_side_entry<M>(p, m, e, cd, user);
    }
    if (tid == 0 && p.spec[3]) atomicOr(p.flags, CO3_FLAG_INEXACT);        // the list did not hold them all
}
