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
// Work item = (user, chunk).  Blocks are persistent and claim items in order through an atomic
// ticket, so the grid as a whole sweeps one window of memory (with a fixed assignment of items to
// blocks the blocks drift apart and a plain streaming kernel loses ~10 % of the bandwidth).  The
// histogram lives in shared memory (one copy per warp, two sets used alternately) and is flushed
// with 64-bit global atomics (spread over several global copies) when the block leaves a segment;
// the moments are reduced in a fixed order per item and stored per item, so the fit does not depend
// on which block converted which item.
//
// Memory pipeline: a thread handles one 4-element vector of g and of m per step (4 steps per
// item).  The loads are asynchronous copies (cp.async, 16 B, L2-only) into thread-private slots of
// a 4-stage shared-memory ring that runs across item boundaries, so three steps (24 KB per block)
// are always in flight without holding registers, and no barrier is needed: a thread only ever
// reads the slots it filled itself, after cp.async.wait_group.
//
// Third variant (fully lagged code, where the header of the iteration is known beforehand):
// the pass also looks every symbol's codeword up and packs it, so the symbols never go to memory.
// A warp's step covers exactly one sub-chunk (128 consecutive elements, four per lane): the lane
// merges its four codewords into one piece, a warp scan places the pieces inside the sub-chunk,
// the pieces are ORed into the warp's own shared-memory slot, and the slot's words go straight to
// the sub-chunk's place in a staging buffer (64 words per sub-chunk) together with the sub-chunk's
// bit count.  No block barrier is involved.  Where a sub-chunk lands in the user's payload depends
// on all earlier ones, so a scan and a concatenation pass follow (co3_encode.cu).
//
// Fourth variant (bias from the current iteration's own moments, t >= 1): the pass runs under the
// previous iteration's bias and only makes sure that every element could be converted again from what it
// stores; reconvert_kernel below does that for the layers whose bias comes out different.  The
// statistics pass that the printed order of Algorithm 1 puts in front of the conversion (stats_kernel)
// then runs at t = 0 only.
#include "co3_internal.h"
#include "co3_quant.cuh"

namespace {

constexpr int STEPS = CO3_TILE / (4 * CO3_THREADS);   // vectors per thread per item (4)
constexpr int STAGES = 4;                             // ring depth of the asynchronous copies

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// Conversion under a guessed bias: an element that the re-conversion pass could not rebuild bit for bit
// from its symbol and its new memory is kept on the side.  Only an element far beyond the largest grid
// value `top` can be one: below top, q is a rounding of a at a quantum of at least ulp(a), so a - q is a
// multiple of ulp(a) no larger than a, hence exact; and a - top is exact while |a| < 2^24 * (lowest
// set bit of top), which 2^(23 - M) * top stays below.  Everything at or above that bound goes on the list.
__device__ __noinline__ void side_push(int32_t* spec, Co3Side* side, uint32_t item, uint32_t pos, uint32_t a_bits) {
    const int k = atomicAdd(spec + 2, 1);
    if (k < CO3_SIDE_CAP) {
        Co3Side e;
        e.item = item; e.pos = pos; e.a_bits = a_bits; e.pad_ = 0;
        side[k] = e;
    } else {
        spec[3] = 1;
    }
}

// a = g + gamma m for the four elements of a vector; moments of the finite ones; NaN/Inf are
// counted and replaced by 0 (so they are coded as +0 and their memory is reset to 0).
// far_bits: 0x7F800000, or (FAR) the bound above which a finite element goes on the side list as well.
template <bool FAR = false>
__device__ __forceinline__ void ef_add4(const float4& gv, const float4& mv, float gamma, float a[4],
                                        double& s1, double& s2, uint32_t& nf, uint32_t far_bits = 0x7F800000u,
                                        int32_t* spec = nullptr, Co3Side* side = nullptr, uint32_t item = 0, uint32_t pos0 = 0,
                                        uint32_t in_mask = 15u) {
    a[0] = __fadd_rn(gv.x, __fmul_rn(gamma, mv.x));
    a[1] = __fadd_rn(gv.y, __fmul_rn(gamma, mv.y));
    a[2] = __fadd_rn(gv.z, __fmul_rn(gamma, mv.z));
    a[3] = __fadd_rn(gv.w, __fmul_rn(gamma, mv.w));
    const uint32_t big = max(max(__float_as_uint(a[0]) & 0x7FFFFFFFu, __float_as_uint(a[1]) & 0x7FFFFFFFu),
                             max(__float_as_uint(a[2]) & 0x7FFFFFFFu, __float_as_uint(a[3]) & 0x7FFFFFFFu));
    if (big >= (FAR ? far_bits : 0x7F800000u)) {   // rare: some element is NaN or Inf (or far out)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t ab = __float_as_uint(a[e]) & 0x7FFFFFFFu;
            if (ab >= 0x7F800000u) { a[e] = 0.0f; ++nf; }
            else if (FAR && ab >= far_bits && ((in_mask >> e) & 1u))
                side_push(spec, side, item, pos0 + e, __float_as_uint(a[e]));
        }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const double ad = (double)fabsf(a[e]);
        s1 += ad;
        s2 = __fma_rn(ad, ad, s2);            // ad*ad is exact in double, so this rounds once
    }
}

struct ItemCtx {                  // what a step needs to know about its item
    const float* gp;              // this thread's first vector of the item's tile (g, m, symbols)
    float* mp;
    uint8_t* sp;
    int lo, hi, seg;              // the item's elements within the tile; its segment
    int user;
    int sub0;                     // index of the chunk's first sub-chunk in the user's sub_bits row
    bool whole;                   // the item covers its whole tile: no edge handling
};

constexpr int SLOT_W = CO3_SUB_WORDS + 2;             // words of a sub-chunk slot (+2: a piece may spill over)

struct PackSmem {                                     // only the packing variant has this
    uint32_t enc[2][CO3_MAXSYM];                      // codeword | length << 16 of this / the next item's segment
    uint32_t slot[CO3_THREADS / 32][SLOT_W];          // one sub-chunk being packed per warp
};

// OR a piece of at most 64 bits into a zero-initialised shared bit image at bit position pos.
__device__ __forceinline__ void or_piece(uint32_t* img, uint32_t pos, unsigned long long v) {
    const uint32_t wi = pos >> 5, sh = pos & 31u;
    const uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
    const uint32_t w0 = lo << sh;
    const uint32_t w1 = __funnelshift_l(lo, hi, sh);  // sh in [0, 31]
    const uint32_t w2 = sh ? (hi >> (32u - sh)) : 0u;
    if (w0) atomicOr(&img[wi], w0);
    if (w1) atomicOr(&img[wi + 1], w1);
    if (w2) atomicOr(&img[wi + 2], w2);
}

// MODE 1: convert, symbols to memory.  MODE 2: convert and pack.  MODE 3: as 1 under a GUESSED bias (that
// of the previous iteration, while the bias of this one is still to come out of this very pass's moments):
// the elements that could not be rebuilt from what is stored are kept, see reconvert_kernel.  (The
// statistics pass has a kernel of its own, below.)
template <int M, int MODE>
__global__ void __launch_bounds__(CO3_THREADS, 4)
ef_kernel(Co3Dev p, const float* __restrict__ g, float* __restrict__ m, uint16_t* __restrict__ sub_bits) {
    static_assert(MODE == 1 || MODE == 2 || MODE == 3, "the statistics pass is stats_kernel");
    constexpr bool PACK = MODE == 2, GUESS = MODE == 3;
    extern __shared__ __align__(16) float4 s_ring[];            // [STAGES][2][CO3_THREADS] (+ PackSmem)
    __shared__ uint32_t s_hist[2][CO3_THREADS / 32][CO3_MAXSYM];   // [item parity][warp][symbol]
    __shared__ double s_red[2][2][CO3_THREADS / 32];
    __shared__ uint32_t s_rednf[2][CO3_THREADS / 32];
    __shared__ uint32_t s_ticket[2];
    __shared__ Co3Chunk s_chunk[2];                   // descriptor of the chunk of s_ticket[.]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // (a launch may cover only the users [u_base, u_base + u_count): the gradient pointer is then that
    // tile's, everything else is indexed by the user's number in the plan)
    const uint32_t n_items = (uint32_t)p.n_chunks * (uint32_t)p.u_count;
    const uint32_t item_base = (uint32_t)p.n_chunks * (uint32_t)p.u_base;
    const uint32_t n_chunks = (uint32_t)p.n_chunks;
    constexpr int VSTRIDE = 4 * CO3_THREADS;          // elements between a thread's vectors

    // Items are claimed through an atomic ticket, two ahead of the one being converted (the copy
    // ring needs the next item's addresses).  Tickets are handed out in item order, so at any time
    // the blocks of the grid work on neighbouring chunks -- the whole GPU sweeps one window of each
    // array like a streaming copy -- and no block falls behind as it does with a fixed assignment.
    if (tid == 0) {
        s_ticket[0] = atomicAdd(p.ticket, 1u);
        s_ticket[1] = atomicAdd(p.ticket, 1u);
    }
    for (int i = tid; i < 2 * (CO3_THREADS / 32) * CO3_MAXSYM; i += CO3_THREADS) (&s_hist[0][0][0])[i] = 0;
    PackSmem& pk = *reinterpret_cast<PackSmem*>(s_ring + STAGES * 2 * CO3_THREADS);
    if (PACK)
        for (int i = tid; i < (CO3_THREADS / 32) * SLOT_W; i += CO3_THREADS) (&pk.slot[0][0])[i] = 0;
    __syncthreads();
    uint32_t item = s_ticket[0], nitem = s_ticket[1];
    if (item >= n_items) return;
    __syncthreads();                                  // both tickets read before slot 0 is reused

    auto make_ctx = [&](uint32_t t, const Co3Chunk& cd) {
        const uint32_t ul = t / n_chunks, uu = ul + (uint32_t)p.u_base;
        ItemCtx x;
        const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
        x.gp = g + (size_t)ul * p.ld + tb + 4 * tid;
        x.mp = m + (size_t)uu * p.ld + tb + 4 * tid;
        x.sp = p.sym + (size_t)uu * p.sld + tb + 4 * tid;
        x.lo = (int)(cd.start - tb);
        x.hi = x.lo + cd.len;
        x.seg = cd.seg;
        x.user = (int)uu;
        x.sub0 = cd.sub0;
        x.whole = cd.len == CO3_TILE;
        return x;
    };
    const uint32_t ring_g = (uint32_t)__cvta_generic_to_shared(s_ring + tid);
    const uint32_t ring_m = (uint32_t)__cvta_generic_to_shared(s_ring + CO3_THREADS + tid);
    constexpr uint32_t SLOT_BYTES = 2 * CO3_THREADS * sizeof(float4);
    static_assert(STAGES == STEPS, "step r of every item lives in ring slot r");

    // one asynchronous step: vector r of item x into ring slot r (one commit group per step)
    auto issue = [&](const ItemCtx& x, bool valid, int r) {
        const int e0 = 4 * tid + VSTRIDE * r;
        if (valid && (x.whole || (e0 < x.hi && e0 + 4 > x.lo))) {
            cp_async16(ring_g + r * SLOT_BYTES, x.gp + VSTRIDE * r);
            cp_async16(ring_m + r * SLOT_BYTES, x.mp + VSTRIDE * r);
        }
        cp_async_commit();
    };

    ItemCtx cur = make_ctx(item, p.chunks[item % n_chunks]);
    issue(cur, true, 0);
    issue(cur, true, 1);
    issue(cur, true, 2);
    bool has_nxt = nitem < n_items;
    ItemCtx nxt = cur;
    if (has_nxt) nxt = make_ctx(nitem, p.chunks[nitem % n_chunks]);

    // the code table of an item's segment is fetched while the previous item is converted
    auto enc_entry = [&](int seg) {
        bool bad = false;
        const int row = co3_row_of(p.hdr_cur[seg], &bad);
        return p.cb.enc[(size_t)row * CO3_MAXSYM + tid];
    };
    if (PACK) {
        pk.enc[0][tid] = enc_entry(cur.seg);
        __syncthreads();
    }
    int cur_seg = -1, par = 0, hpar = 0;
    unsigned long long* hist_copy = p.hist + (size_t)(blockIdx.x % (unsigned)p.hist_copies) * p.S * CO3_MAXSYM;
    QParams q;
    q.top = 0.0f; q.low_bits = 0; q.e0 = 0; q.far_bits = 0x7F800000u;

    while (true) {
        // thread 0 claims the item after next now, fetches its chunk descriptor half-way through the
        // item and publishes both before the item's barrier: no thread ever waits for either
        uint32_t claim = n_items;
        Co3Chunk claim_cd;
        if (tid == 0 && has_nxt) claim = atomicAdd(p.ticket, 1u);
        if (cur.seg != cur_seg) {
            cur_seg = cur.seg;
            const int lambda = p.bias_cur[cur.seg] + p.cF;
            q.top = __fmul_rn((float)p.Kmax, pow2f(lambda));
            q.low_bits = __float_as_uint(pow2f(lambda + M));
            q.e0 = (uint32_t)(lambda + 150);
            q.far_bits = min(__float_as_uint(q.top) + ((23u - M) << 23), 0x7F800000u);   // top < 2^100: no overflow into the sign
        }
        uint32_t enc_next = 0;                        // PACK: my entry of the next item's code table
        if (PACK && has_nxt) enc_next = enc_entry(nxt.seg);
        const uint32_t* enc_tab = pk.enc[par];
        // PACK: this lane's word of the warp's slot, of the sub-chunk's staging slot (step 0), the
        // lane-31 pointer into sub_bits, the chunk's sub-chunk range, the warp's share of its bits
        uint32_t* slot_l = pk.slot[warp] + lane;
        uint32_t* pk_stage = PACK ? p.slot_buf + ((size_t)item * (CO3_TILE / CO3_SUB) + warp) * CO3_SUB_WORDS + lane : nullptr;
        const int pk_sub_first = cur.lo / CO3_SUB, pk_sub_last = (cur.hi - 1) / CO3_SUB;
        uint16_t* pk_sb = PACK ? sub_bits + (size_t)cur.user * p.n_sub + cur.sub0 + (warp - pk_sub_first) : nullptr;
        uint32_t chunk_bits_w = 0;
        double s1 = 0.0, s2 = 0.0;
        uint32_t nf = 0;
#pragma unroll
        for (int r = 0; r < STEPS; ++r) {
            // the producer is always STAGES - 1 = 3 steps ahead: step 3 of this item, then steps
            // 0..2 of the next one, each into the slot the consumer has just left
            if (r == 0) issue(cur, true, 3);
            else issue(nxt, has_nxt, r - 1);
            if (r == 2 && tid == 0 && claim < n_items) claim_cd = p.chunks[claim % n_chunks];
            cp_async_wait<STAGES - 1>();              // this step's copies have landed
            const uint32_t slot = r * SLOT_BYTES;
            const int e0 = 4 * tid + VSTRIDE * r;
            const bool full = cur.whole || ((e0 >= cur.lo) && (e0 + 4 <= cur.hi));
            const bool some = full || (e0 < cur.hi && e0 + 4 > cur.lo);
            unsigned long long piece = 0;             // PACK: this lane's four codewords, merged
            uint32_t plen = 0;
            if (some) {
                float4 gv = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(s_ring + tid) + slot);
                float4 mv = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(s_ring + CO3_THREADS + tid) + slot);
                float a[4], mo[4];
                uint32_t so[4], en[4] = {0u, 0u, 0u, 0u};
                if (full) {
                    if (GUESS) ef_add4<true>(gv, mv, p.gamma, a, s1, s2, nf, q.far_bits, p.spec, p.side, item_base + item, (uint32_t)e0, 15u);
                    else ef_add4(gv, mv, p.gamma, a, s1, s2, nf);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        quantize<M>(a[e], q, so[e], mo[e]);
                        atomicAdd(&s_hist[hpar][warp][so[e]], 1u);
                        if (PACK) en[e] = enc_tab[so[e]];
                    }
                    *reinterpret_cast<float4*>(cur.mp + VSTRIDE * r) = make_float4(mo[0], mo[1], mo[2], mo[3]);
                    if (!PACK)
                        *reinterpret_cast<uint32_t*>(cur.sp + VSTRIDE * r) = so[0] | (so[1] << 8) | (so[2] << 16) | (so[3] << 24);
                } else {                              // a vector on the chunk's edge: element by element
                    const bool in0 = e0 >= cur.lo && e0 < cur.hi, in1 = e0 + 1 >= cur.lo && e0 + 1 < cur.hi;
                    const bool in2 = e0 + 2 >= cur.lo && e0 + 2 < cur.hi, in3 = e0 + 3 >= cur.lo && e0 + 3 < cur.hi;
                    const bool in[4] = {in0, in1, in2, in3};
                    if (!in0) { gv.x = 0.0f; mv.x = 0.0f; }   // elements of the neighbouring chunk count as 0
                    if (!in1) { gv.y = 0.0f; mv.y = 0.0f; }
                    if (!in2) { gv.z = 0.0f; mv.z = 0.0f; }
                    if (!in3) { gv.w = 0.0f; mv.w = 0.0f; }
                    if (GUESS) ef_add4<true>(gv, mv, p.gamma, a, s1, s2, nf, q.far_bits, p.spec, p.side, item_base + item, (uint32_t)e0,
                                             (uint32_t)in0 | ((uint32_t)in1 << 1) | ((uint32_t)in2 << 2) | ((uint32_t)in3 << 3));
                    else ef_add4(gv, mv, p.gamma, a, s1, s2, nf);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (in[e]) {
                            quantize<M>(a[e], q, so[e], mo[e]);
                            atomicAdd(&s_hist[hpar][warp][so[e]], 1u);
                            cur.mp[VSTRIDE * r + e] = mo[e];
                            if (PACK) en[e] = enc_tab[so[e]];
                            else cur.sp[VSTRIDE * r + e] = (uint8_t)so[e];
                        }
                    }
                }
                if (PACK) {                           // an element outside the chunk has entry 0: no bits
                    const uint32_t l0 = en[0] >> 16, l2 = en[2] >> 16;
                    const uint32_t c01 = (en[0] & 0xFFFFu) | ((en[1] & 0xFFFFu) << l0);
                    const uint32_t c23 = (en[2] & 0xFFFFu) | ((en[3] & 0xFFFFu) << l2);
                    const uint32_t l01 = l0 + (en[1] >> 16);
                    piece = (unsigned long long)c01 | ((unsigned long long)c23 << l01);
                    plen = l01 + l2 + (en[3] >> 16);
                }
            }
            if (PACK) {
                // this warp's step is sub-chunk 8 r + warp: place the lane's piece after those of the
                // lanes below, OR it into the warp's slot, then move the slot's words to the staging
                // buffer (and leave the slot zero for the next step)
                uint32_t x = plen;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
                    if (lane >= o) x += y;
                }
                constexpr int SC_STEP = CO3_THREADS / 32;           // sub-chunk of this step: SC_STEP * r + warp
                if (plen) or_piece(pk.slot[warp], x - plen, piece);
                const uint32_t total = __shfl_sync(0xffffffffu, x, 31);
                chunk_bits_w += total;
                __syncwarp();
                if (32u * lane < total) {
                    pk_stage[SC_STEP * r * CO3_SUB_WORDS] = *slot_l;
                    *slot_l = 0;
                }
                if (total > 1024u) {                                // rare: above 8 bits per symbol
                    if (32u * (lane + 32) < total) {
                        pk_stage[SC_STEP * r * CO3_SUB_WORDS + 32] = slot_l[32];
                        slot_l[32] = 0;
                    }
                }
                if (lane == 31 && SC_STEP * r + warp >= pk_sub_first && SC_STEP * r + warp <= pk_sub_last)
                    pk_sb[SC_STEP * r] = (uint16_t)total;
                __syncwarp();
            }
        }
        if (PACK && lane == 31) atomicAdd(&p.chunk_bits[item], chunk_bits_w);   // cleared before the launch
        // this item's moments, reduced in a fixed order (lanes, then warps) and stored per item:
        // the fit does not depend on which block converted which item
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s1 += __shfl_down_sync(0xffffffffu, s1, o);
            s2 += __shfl_down_sync(0xffffffffu, s2, o);
            nf += __shfl_down_sync(0xffffffffu, nf, o);
        }
        if (lane == 0) { s_red[par][0][warp] = s1; s_red[par][1][warp] = s2; s_rednf[par][warp] = nf; }
        if (tid == 0) {
            s_ticket[par] = claim;
            if (claim < n_items) s_chunk[par] = claim_cd;
        }
        if (PACK) pk.enc[par ^ 1][tid] = enc_next;
        __syncthreads();                              // sums, histogram, claim (and the next code table)
        if (tid == 0) {
            double t1 = 0.0, t2 = 0.0;
            uint32_t tn = 0;
#pragma unroll
            for (int w = 0; w < CO3_THREADS / 32; ++w) { t1 += s_red[par][0][w]; t2 += s_red[par][1][w]; tn += s_rednf[par][w]; }
            const uint32_t pi = item_base + item;
            p.part_s1[pi] = t1; p.part_s2[pi] = t2; p.part_nf[pi] = tn;
        }
        // When the block leaves the segment (or ends) its histogram goes to global memory; the next
        // item counts in the other copy, and this copy is not touched again before a later barrier.
        // (Flushing after every item instead costs a single-segment E4M3 gradient 30 % of the pass:
        // all blocks then hammer the same 256 counters.)
        if (!has_nxt || nxt.seg != cur.seg) {
            if (tid < p.nsym) {
                unsigned long long tot = 0;
#pragma unroll
                for (int w = 0; w < CO3_THREADS / 32; ++w) { tot += s_hist[hpar][w][tid]; s_hist[hpar][w][tid] = 0; }
                if (tot) atomicAdd(&hist_copy[(size_t)cur.seg * CO3_MAXSYM + tid], tot);
            }
            hpar ^= 1;
        }
        if (!has_nxt) break;
        item = nitem;
        cur = nxt;
        nitem = s_ticket[par];
        has_nxt = nitem < n_items;
        if (has_nxt) nxt = make_ctx(nitem, s_chunk[par]);
        par ^= 1;
    }
    cp_async_wait<0>();
}

// Statistics pass (the bias of Algorithm 1 line 8 taken from the moments of g_t + gamma m_{t-1}
// themselves, before they are converted): nothing is written but three numbers per item, so a plain
// grid does it -- one block per item, all of a thread's eight 128-bit loads in flight at once, five
// blocks per SM so that nobody waits for the reduction at the end.  The block scheduler hands the
// items out in order, which keeps the sweep of a streaming read.  The loads are marked evict-first
// (read once: 117 -> 110 us on 8 x 11.2 M elements), except those of the items the convert pass will
// take first, which ask to stay in L2.  The items are walked from the last one down, so the pass ends
// with exactly those, and begins where the previous iteration's convert pass ended.
// A thread takes the same elements in the same order as in the convert pass and the partial sums are
// combined in the same order, so both passes give the same bits.
constexpr uint32_t STATS_KEEP_ITEMS = (32u << 20) / (2 * sizeof(float) * CO3_TILE);   // 32 MB of g and m

__device__ __forceinline__ float4 ld_keep(const float4* ptr, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr), "l"(policy));
    return v;
}

__global__ void __launch_bounds__(CO3_THREADS, 4)
stats_kernel(Co3Dev p, const float* __restrict__ g, const float* __restrict__ m) {
    __shared__ double s_red[2][CO3_THREADS / 32];
    __shared__ uint32_t s_rednf[CO3_THREADS / 32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_chunks = (uint32_t)p.n_chunks;
    const uint32_t it = gridDim.x - 1u - blockIdx.x;          // item: user (of this launch) x chunk
    const uint32_t ul = it / n_chunks, uu = ul + (uint32_t)p.u_base;
    const Co3Chunk cd = p.chunks[it - ul * n_chunks];
    const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
    const int lo = (int)(cd.start - tb), hi = lo + cd.len;
    const bool whole = cd.len == CO3_TILE;
    constexpr int VSTRIDE = 4 * CO3_THREADS;
    const float4* gp = reinterpret_cast<const float4*>(g + (size_t)ul * p.ld + tb + 4 * tid);
    const float4* mp = reinterpret_cast<const float4*>(m + (size_t)uu * p.ld + tb + 4 * tid);
    const bool keep = it < STATS_KEEP_ITEMS;
    uint64_t keep_policy = 0;
    if (keep) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep_policy));
    float4 gv[STEPS], mv[STEPS];
#pragma unroll
    for (int r = 0; r < STEPS; ++r) {
        const int e0 = 4 * tid + VSTRIDE * r;
        gv[r] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        mv[r] = gv[r];
        if (whole || (e0 < hi && e0 + 4 > lo)) {
            if (keep) {
                gv[r] = ld_keep(gp + (VSTRIDE / 4) * r, keep_policy);
                mv[r] = ld_keep(mp + (VSTRIDE / 4) * r, keep_policy);
            } else {
                gv[r] = __ldcs(gp + (VSTRIDE / 4) * r);
                mv[r] = __ldcs(mp + (VSTRIDE / 4) * r);
            }
        }
    }
    double s1 = 0.0, s2 = 0.0;
    uint32_t nf = 0;
#pragma unroll
    for (int r = 0; r < STEPS; ++r) {
        const int e0 = 4 * tid + VSTRIDE * r;
        if (!whole && !(e0 >= lo && e0 + 4 <= hi)) {          // a vector on the chunk's edge, or outside it
            if (e0 + 4 <= lo || e0 >= hi) continue;
            if (e0 < lo || e0 >= hi) { gv[r].x = 0.0f; mv[r].x = 0.0f; }   // elements of the neighbouring chunk count as 0
            if (e0 + 1 < lo || e0 + 1 >= hi) { gv[r].y = 0.0f; mv[r].y = 0.0f; }
            if (e0 + 2 < lo || e0 + 2 >= hi) { gv[r].z = 0.0f; mv[r].z = 0.0f; }
            if (e0 + 3 < lo || e0 + 3 >= hi) { gv[r].w = 0.0f; mv[r].w = 0.0f; }
        }
        float a[4];
        ef_add4(gv[r], mv[r], p.gamma, a, s1, s2, nf);
    }
    // lanes, then warps, in the order of the convert pass
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_down_sync(0xffffffffu, s1, o);
        s2 += __shfl_down_sync(0xffffffffu, s2, o);
        nf += __shfl_down_sync(0xffffffffu, nf, o);
    }
    if (lane == 0) { s_red[0][warp] = s1; s_red[1][warp] = s2; s_rednf[warp] = nf; }
    __syncthreads();
    if (tid == 0) {
        double t1 = 0.0, t2 = 0.0;
        uint32_t tn = 0;
#pragma unroll
        for (int w = 0; w < CO3_THREADS / 32; ++w) { t1 += s_red[0][w]; t2 += s_red[1][w]; tn += s_rednf[w]; }
        const uint32_t pi = n_chunks * (uint32_t)p.u_base + it;
        p.part_s1[pi] = t1; p.part_s2[pi] = t2; p.part_nf[pi] = tn;
    }
}

// Bias from the current moments WITHOUT a statistics pass in every iteration.  The convert pass runs
// under a guess (the previous iteration's bias), the fit that follows it finds the bias of this
// iteration from the pass's own moments -- the same sums, in the same order, that a statistics pass
// would have handed it -- and lists the layers where the two differ.  Those layers (usually none, and
// if any, small ones whose fit is noisy) are converted again here: a = g + gamma m is rebuilt from
// what the first conversion stored, a = q + m' (exact: the residual identity of Algorithm 1 line 10
// read backwards; the few elements so far out that it does not hold were kept on a side list by the
// convert pass), and quantised at the right bias: symbols, memory and histogram are then bit for bit
// what the statistics-pass-first order of Algorithm 1 line 8 gives.
// Grid: a few blocks per SM; a block that finds the list empty returns at once.  The last block to
// finish applies the side list and clears the counters for the next iteration.
template <int M>
__global__ void __launch_bounds__(CO3_THREADS)
reconvert_kernel(Co3Dev p, float* __restrict__ m) {
    __shared__ uint32_t s_hist[2][CO3_MAXSYM];        // symbols taken out of the layer's histogram, symbols put in
    __shared__ int s_last;
    const int tid = threadIdx.x;
    const int n = p.spec[0];
    if (n == 0) {                                     // every guess was right
        if (blockIdx.x == 0 && tid == 0) { p.spec[2] = 0; p.spec[3] = 0; }
        return;
    }
    for (int k = 0; k < n; ++k) {
        const int seg = p.redo_seg[k];
        const int c0 = p.seg_chunk0[seg], nck = p.seg_chunk0[seg + 1] - c0;
        if ((int64_t)blockIdx.x >= (int64_t)nck * p.U) continue;    // (uniform in the block)
        redo_items<M>(p, m, seg, c0, nck, p.redo_old[k], p.bias_cur[seg], blockIdx.x, gridDim.x, tid, CO3_THREADS, s_hist);
    }
    // the last block to get here: side list, then the counters
    __threadfence();
    if (tid == 0) s_last = atomicAdd(p.spec + 1, 1) == (int)gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const int n_side = min(p.spec[2], CO3_SIDE_CAP);
    for (int j = tid; j < n_side; j += CO3_THREADS) {
        const Co3Side e = p.side[j];
        const uint32_t user = e.item / (uint32_t)p.n_chunks;
        const Co3Chunk cd = p.chunks[e.item - user * (uint32_t)p.n_chunks];
        bool listed = false;
        for (int k = 0; k < n; ++k) listed |= p.redo_seg[k] == cd.seg;
        if (listed) redo_side_entry<M>(p, m, e, cd, user);   // (a layer that kept the guess: what is stored is right)
    }
    if (tid == 0) {
        if (p.spec[3]) atomicOr(p.flags, CO3_FLAG_INEXACT);   // more far-out elements than the list holds, and a wrong guess
        p.spec[0] = 0; p.spec[1] = 0; p.spec[2] = 0; p.spec[3] = 0;
    }
}

// Inspection: copy the stored symbols to a caller buffer [U][d] in the public form.
__global__ void symbol_export_kernel(Co3Dev p, uint8_t* __restrict__ out) {
    const int64_t n = (int64_t)p.U * p.d;
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += (int64_t)gridDim.x * blockDim.x) {
        const int64_t u = k / p.d, i = k - u * p.d;
        out[k] = (uint8_t)co3_sym_public(p.sym[(size_t)u * p.sld + i], p.nm);
    }
}

typedef void (*ef_fn)(Co3Dev, const float*, float*, uint16_t*);
constexpr size_t RING_BYTES = (size_t)STAGES * 2 * CO3_THREADS * sizeof(float4);

template <int MODE>
ef_fn pick_kernel(int M) {
    switch (M) {
        case 1: return ef_kernel<1, MODE>;
        case 2: return ef_kernel<2, MODE>;
        case 3: return ef_kernel<3, MODE>;
        case 4: return ef_kernel<4, MODE>;
        case 5: return ef_kernel<5, MODE>;
        default: return ef_kernel<6, MODE>;
    }
}

int ef_grid(const co3_plan* pl, ef_fn fn, size_t smem) {
    int n = 0;
    // static + dynamic shared memory exceed the 48 KiB default, so the kernel has to opt in
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        (void)cudaGetLastError();
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, CO3_THREADS, smem);
    if (n < 1) n = 1;
    const int64_t items = pl->dev.n_chunks * (int64_t)pl->dev.U;
    const int64_t grid = (int64_t)pl->num_sms * n;
    return (int)(items < grid ? items : grid);
}

}  // namespace

cudaError_t co3_launch_symbol_export(co3_plan* pl, uint8_t* symbols, cudaStream_t st) {
    symbol_export_kernel<<<pl->num_sms * 8, 256, 0, st>>>(pl->dev, symbols);
    return cudaGetLastError();
}

// u_base / u_count: the users this launch covers (g is then the gradient of those users only).
cudaError_t co3_launch_stats(co3_plan* pl, const float* g, const float* m, int u_base, int u_count, cudaStream_t st) {
    Co3Dev p = pl->dev;
    p.u_base = u_base; p.u_count = u_count;
    const int64_t items = p.n_chunks * (int64_t)u_count;       // below 2^31 (checked when the plan is made)
    co3_prof_begin(pl, CO3_K_STATS, st);
    stats_kernel<<<(unsigned)items, CO3_THREADS, 0, st>>>(p, g, m);
    co3_prof_end(pl, CO3_K_STATS, st, 1);
    return cudaGetLastError();
}

// first: this launch starts the iteration's histogram (later tiles of the same iteration add to it)
// cleared: the fit kernel launched just before has zeroed the histogram and the ticket
cudaError_t co3_launch_convert(co3_plan* pl, const float* g, float* m, int u_base, int u_count, bool first,
                               cudaStream_t st, bool cleared, bool check_guess) {
    // one memset clears the histogram and the item ticket that follows it in the same allocation
    cudaError_t e = cudaSuccess;
    if (cleared) {}
    else if (first) e = cudaMemsetAsync(pl->dev.hist, 0, sizeof(unsigned long long) * ((size_t)pl->dev.hist_copies * pl->dev.S * CO3_MAXSYM + 1), st);
    else e = cudaMemsetAsync(pl->dev.ticket, 0, sizeof(unsigned int), st);
    if (e != cudaSuccess) return e;
    ef_fn fn = check_guess ? pick_kernel<3>(pl->dev.M) : pick_kernel<1>(pl->dev.M);
    int& grid = check_guess ? pl->grid_convert_spec : pl->grid_convert;
    if (!grid) grid = ef_grid(pl, fn, RING_BYTES);
    Co3Dev p = pl->dev;
    p.u_base = u_base; p.u_count = u_count;
    const int64_t items = p.n_chunks * (int64_t)u_count;
    co3_prof_begin(pl, CO3_K_CONVERT, st);
    fn<<<(int)(items < grid ? items : grid), CO3_THREADS, RING_BYTES, st>>>(p, g, m, nullptr);
    co3_prof_end(pl, CO3_K_CONVERT, st, 1);
    return cudaGetLastError();
}

typedef void (*reconv_fn)(Co3Dev, float*);
cudaError_t co3_launch_reconvert(co3_plan* pl, float* m, cudaStream_t st) {
    reconv_fn fn;
    switch (pl->dev.M) {
        case 1: fn = reconvert_kernel<1>; break;
        case 2: fn = reconvert_kernel<2>; break;
        case 3: fn = reconvert_kernel<3>; break;
        case 4: fn = reconvert_kernel<4>; break;
        case 5: fn = reconvert_kernel<5>; break;
        default: fn = reconvert_kernel<6>; break;
    }
    const int64_t items = pl->dev.n_chunks * (int64_t)pl->dev.U, grid = (int64_t)pl->num_sms * 4;
    co3_prof_begin(pl, CO3_K_RECONVERT, st);
    fn<<<(int)(items < grid ? items : grid), CO3_THREADS, 0, st>>>(pl->dev, m);
    co3_prof_end(pl, CO3_K_RECONVERT, st, 1);
    return cudaGetLastError();
}

// Fully lagged code: convert and pack in one pass (chunk images go to the plan's staging slots).
cudaError_t co3_launch_convert_pack(co3_plan* pl, const float* g, float* m, uint16_t* sub_bits, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(pl->dev.hist, 0, sizeof(unsigned long long) * ((size_t)pl->dev.hist_copies * pl->dev.S * CO3_MAXSYM + 1), st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(pl->dev.chunk_bits, 0, sizeof(uint32_t) * (size_t)pl->dev.n_chunks * pl->dev.U, st);
    if (e != cudaSuccess) return e;
    constexpr size_t smem = RING_BYTES + sizeof(PackSmem);
    ef_fn fn = pick_kernel<2>(pl->dev.M);
    if (!pl->grid_convert) pl->grid_convert = ef_grid(pl, fn, smem);
    co3_prof_begin(pl, CO3_K_CONVERT, st);
    fn<<<pl->grid_convert, CO3_THREADS, smem, st>>>(pl->dev, g, m, sub_bits);
    co3_prof_end(pl, CO3_K_CONVERT, st, 1);
    return cudaGetLastError();
}
