// h_Hf on the device (Algorithm 1 line 9): Huffman-code the converted symbols of every user
// into the chunked container, in ONE launch (enc_single_kernel).
// Work item = (user, chunk) = one block of 64 threads.  The chunk's tile is cut into 256 runs of 16
// symbols; thread t owns the runs t, t + 64, t + 128, t + 192, so that a warp's 128-bit symbol loads
// are contiguous and the places where neighbouring lanes later write into the chunk image lie a few
// words apart (distinct banks) instead of a whole granule apart.  Every symbol is looked up ONCE
// (packed codeword + length): a run's 16 codewords are merged pairwise in registers into four pieces
// of at most 64 bits, and the pieces of all four runs stay in registers while the block scans the run
// lengths into bit offsets (which also gives the sub-chunk lengths and the chunk size); then the
// pieces are ORed into a shared-memory image of the chunk, the block learns the chunk's offset in the
// user's payload from the sizes the earlier chunks have published (see below) and stores the image
// with 128-bit accesses.
// Bound: the load/store data pipe of the SM (one table look-up per symbol in random banks, the ORs
// into the image) and issue slots; HBM traffic is small (1 B/element read, ~0.87 B/element written).
//
// The fully lagged-code mode uses enc_scan_kernel and enc_concat_kernel instead (the symbols were
// packed per sub-chunk by the convert pass).
#include "co3_internal.h"

namespace {

constexpr int RUN = 16;                                 // symbols per run (one 128-bit load)
constexpr int BUF_WORDS = CO3_TILE * CO3_MAXLEN / 32;   // 2048: a chunk at 16 bits per symbol
static_assert(CO3_SUB == 8 * RUN, "eight runs are a sub-chunk");

// chunk_off[u][c] = exclusive prefix of the chunk word counts of user u; one block per user.
// Used by the fully lagged code only: the convert-and-pack pass added up the code bits of each chunk;
// the word counts are derived here and stored for the concatenation pass.
__global__ void __launch_bounds__(1024)
enc_scan_kernel(Co3Dev p, uint32_t* __restrict__ chunk_off, unsigned long long* __restrict__ user_bits) {
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_carry;
    __shared__ unsigned long long s_bits[32];
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* in = p.chunk_words + (size_t)u * p.n_chunks;
    uint32_t* inb = p.chunk_bits + (size_t)u * p.n_chunks;
    uint32_t* out = chunk_off + (size_t)u * (p.n_chunks + 1);
    unsigned long long my_bits = 0;                   // r_t^(u): code bits of this user
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < p.n_chunks; base += 1024) {
        const int64_t i = base + tid;
        uint32_t v = 0u;
        if (i < p.n_chunks) {
            const uint32_t bits = inb[i];
            v = 4u * ((bits + 127u) / 128u);
            in[i] = v;
            my_bits += bits;
        }
        uint32_t x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) s_warp[warp] = x;
        __syncthreads();
        if (warp == 0) {
            uint32_t t = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, t, o);
                if (lane >= o) t += y;
            }
            s_warp[lane] = t;
        }
        __syncthreads();
        const uint32_t carry = s_carry;
        const uint32_t excl = carry + (warp ? s_warp[warp - 1] : 0u) + x - v;
        if (i < p.n_chunks) out[i] = excl;
        __syncthreads();
        if (tid == 1023) s_carry = carry + s_warp[31];
        __syncthreads();
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_bits += __shfl_xor_sync(0xffffffffu, my_bits, o);
    if (lane == 0) s_bits[warp] = my_bits;
    __syncthreads();
    if (tid == 0) {
        unsigned long long tb = 0;
        for (int k = 0; k < 32; ++k) tb += s_bits[k];
        user_bits[u] = tb;
        const uint32_t total = s_carry;
        out[p.n_chunks] = total;
        const uint32_t ovf = (int64_t)total > p.cap_words;
        p.user_ovf[u] = ovf;
        if (ovf) atomicOr(p.flags, CO3_FLAG_CAPACITY);
    }
}

// OR a piece of at most 64 bits into the chunk image at bit position pos.
__device__ __forceinline__ void put_piece(uint32_t* s_buf, uint32_t pos, unsigned long long v) {
    const uint32_t wi = pos >> 5, bs = pos & 31u;
    const uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
    const uint32_t w0 = lo << bs;
    const uint32_t w1 = __funnelshift_l(lo, hi, bs);
    const uint32_t w2 = __funnelshift_l(hi, 0u, bs);
    if (w0) atomicOr(&s_buf[wi], w0);
    if (w1) atomicOr(&s_buf[wi + 1], w1);
    if (w2) atomicOr(&s_buf[wi + 2], w2);
}

// ---- single pass: lengths, offsets and packing in one kernel ---------------------------------
// One block per (user, chunk) as above, but the item is a ticket (so every item with a smaller
// number has been claimed by a block that is running or done), and the chunk's word offset is
// summed from what the earlier chunks of the same user PUBLISH: each block stores its own word
// count (a self-validating word) and adds it to the totals of its group of 64 chunks (a 64-bit word:
// arrivals << 56 | payload words << 32 | code bits).  A block needs only such counts, never another block's offset, so
// there is no chain: after packing its chunk into shared memory (by then the earlier blocks have
// long published) it adds up the totals of the complete groups before its own and the counts of
// the earlier chunks of its own group.  Every wait is bounded; a wait that runs out raises
// CO3_FLAG_TIMEOUT and the block writes nothing.
constexpr uint32_t ST_VALID = 0x80000000u;
constexpr int GRP_SHIFT = 6, GRP_SIZE = 1 << GRP_SHIFT;
// (the polls of a word in L2 are limited by Co3Dev::spin_limit: 2^20 of them take about a second)

__device__ __forceinline__ uint32_t wait_count(const uint32_t* st, int spin_limit, bool& timeout) {
    const volatile uint32_t* v = st;
    for (int k = 0; k < spin_limit; ++k) {
        const uint32_t w = *v;
        if (w & ST_VALID) return w & ~ST_VALID;
    }
    timeout = true;
    return 0;
}
// waits until `expect` chunks have arrived in the group; returns words << 32 | bits
__device__ __forceinline__ unsigned long long wait_group(const unsigned long long* grp, uint32_t expect, int spin_limit,
                                                         bool& timeout) {
    const volatile unsigned long long* v = grp;
    for (int k = 0; k < spin_limit; ++k) {
        const unsigned long long w = *v;
        if ((w >> 56) == (unsigned long long)expect) return w & ((1ull << 56) - 1);
    }
    timeout = true;
    return 0;
}

// ENC_THREADS threads per chunk (64 or 128), each owning CO3_TILE / 16 / ENC_THREADS runs.
template <int ENC_THREADS, int MIN_BLOCKS>
__global__ void __launch_bounds__(ENC_THREADS, MIN_BLOCKS)
enc_single_kernel(Co3Dev p, const co3_seg_header* __restrict__ hdr, uint16_t* __restrict__ sub_bits,
                  uint32_t* __restrict__ chunk_off, unsigned long long* __restrict__ user_bits,
                  uint32_t* __restrict__ bitstream, uint32_t n_items) {
    __shared__ __align__(16) uint32_t s_enc[CO3_MAXSYM];            // codeword | length << 16
    __shared__ __align__(16) uint32_t s_buf[BUF_WORDS + 4];         // image of the chunk
    constexpr int ENC_WARPS = ENC_THREADS / 32;
    constexpr int RUNS_PER_THREAD = CO3_TILE / RUN / ENC_THREADS;   // thread t owns runs t + ENC_THREADS * k
    constexpr int NP = RUNS_PER_THREAD / 2;                         // two runs share a word of the scans
    static_assert(RUNS_PER_THREAD % 2 == 0 && ENC_THREADS * 256 <= 65536 && ENC_THREADS >= GRP_SIZE, "see the scan");
    __shared__ uint32_t s_wtot[NP][ENC_WARPS];                      // per warp: bits of its runs 2j | 2j + 1, packed
    __shared__ uint32_t s_sum[ENC_WARPS];
    __shared__ uint32_t s_item;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_item = atomicAdd(p.enc_ticket, 1u);
    __syncthreads();
    const uint32_t item = s_item;
    if (item >= n_items) return;                      // (only a launch that did not start the tickets at 0 gets here)
    bool bad = false;
    struct { uint32_t u, c; Co3Chunk cd; } it;
    {
        const uint32_t n_chunks = (uint32_t)p.n_chunks;
        it.u = item / n_chunks;
        it.c = item - it.u * n_chunks;
        it.cd = p.chunks[it.c];
    }
    const int64_t tb = it.cd.start & ~(int64_t)(CO3_TILE - 1);
    const int tlo = (int)(it.cd.start - tb), thi = tlo + it.cd.len;
    // this thread's runs of 16 symbols (run k = elements 16 (128 k + tid) .. + 15 of the tile)
    uint4 v[RUNS_PER_THREAD];
    uint32_t mask[RUNS_PER_THREAD];
    {
        const uint4* src = reinterpret_cast<const uint4*>(p.sym + (size_t)it.u * p.sld + tb);
#pragma unroll
        for (int k = 0; k < RUNS_PER_THREAD; ++k) {
            const int e0 = RUN * (ENC_THREADS * k + tid);
            const int a = min(max(tlo - e0, 0), RUN), b = max(min(thi - e0, RUN), a);
            mask[k] = ((1u << b) - 1u) & ~((1u << a) - 1u);
            v[k] = mask[k] ? __ldg(src + ENC_THREADS * k + tid) : make_uint4(0, 0, 0, 0);
        }
    }
    {
        const size_t row = (size_t)(p.code_by_segment ? it.cd.seg : co3_row_of(hdr[it.cd.seg], &bad)) * CO3_MAXSYM;
        if (tid < CO3_MAXSYM / 4) reinterpret_cast<uint4*>(s_enc)[tid] = __ldg(reinterpret_cast<const uint4*>(p.cb.enc + row) + tid);
    }
    __syncthreads();
    // one look-up per symbol; 16 codewords -> 8 pieces (<= 32 bits) -> 4 pieces (<= 64 bits), kept in registers
    unsigned long long piece[RUNS_PER_THREAD][4];
    uint32_t plen[RUNS_PER_THREAD];                   // the four piece lengths of a run, one byte each
    uint32_t bits[RUNS_PER_THREAD];                   // code bits of the run
#pragma unroll
    for (int k = 0; k < RUNS_PER_THREAD; ++k) {
        const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
        uint32_t ent[RUN];
        if (mask[k] == 0xFFFFu) {
#pragma unroll
            for (int i = 0; i < RUN; ++i) ent[i] = s_enc[__byte_perm(w[i >> 2], 0, 0x4440 + (i & 3))];
        } else {
#pragma unroll
            for (int i = 0; i < RUN; ++i) {
                const uint32_t e = s_enc[__byte_perm(w[i >> 2], 0, 0x4440 + (i & 3))];
                ent[i] = ((mask[k] >> i) & 1u) ? e : 0u;
            }
        }
        uint32_t c1[8], l1[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t x0 = ent[2 * q], x1 = ent[2 * q + 1];
            c1[q] = (x0 & 0xFFFFu) | ((x1 & 0xFFFFu) << (x0 >> 16));
            l1[q] = (x0 >> 16) + (x1 >> 16);
        }
        plen[k] = 0;
        bits[k] = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            piece[k][q] = (unsigned long long)c1[2 * q] | ((unsigned long long)c1[2 * q + 1] << l1[2 * q]);
            const uint32_t l = l1[2 * q] + l1[2 * q + 1];
            plen[k] |= l << (8 * q);
            bits[k] += l;
        }
    }
    // Bit offsets: the runs follow each other in the order k * ENC_THREADS + tid.  Two runs of a thread
    // share a word of the scan (a run has at most 256 bits, all runs of one k at most 32768).
    uint32_t x[NP], own[NP];
#pragma unroll
    for (int j = 0; j < NP; ++j) own[j] = x[j] = bits[2 * j] | (bits[2 * j + 1] << 16);
    {   // sub-chunk lengths: a sub-chunk is the eight runs of eight neighbouring threads at one k
        uint32_t y[NP];
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            y[j] = x[j];
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) y[j] += __shfl_xor_sync(0xffffffffu, y[j], o);
        }
        if ((tid & 7) == 0) {
            const int sub_first = tlo / CO3_SUB, sub_last = (thi - 1) / CO3_SUB;
            uint16_t* sbp = sub_bits + (size_t)it.u * p.n_sub + it.cd.sub0;
#pragma unroll
            for (int k = 0; k < RUNS_PER_THREAD; ++k) {
                const int sc = (ENC_THREADS / 8) * k + (tid >> 3);
                if (sc >= sub_first && sc <= sub_last) sbp[sc - sub_first] = (uint16_t)((k & 1) ? y[k / 2] >> 16 : y[k / 2] & 0xFFFFu);
            }
        }
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            const uint32_t a = __shfl_up_sync(0xffffffffu, x[j], o);
            if (lane >= o) x[j] += a;
        }
    }
    if (lane == 31) {
#pragma unroll
        for (int j = 0; j < NP; ++j) s_wtot[j][warp] = x[j];
    }
    __syncthreads();
    uint32_t pos[RUNS_PER_THREAD], tot = 0;
#pragma unroll
    for (int j = 0; j < NP; ++j) {
        uint32_t before = 0, all = 0;                 // packed sums of the warps before this one, of all warps
#pragma unroll
        for (int w = 0; w < ENC_WARPS; ++w) {
            const uint32_t t = s_wtot[j][w];
            if (w < warp) before += t;
            all += t;
        }
        const uint32_t excl = x[j] - own[j] + before; // exclusive within k = 2j | within k = 2j + 1
        pos[2 * j] = tot + (excl & 0xFFFFu);
        tot += all & 0xFFFFu;
        pos[2 * j + 1] = tot + (excl >> 16);
        tot += all >> 16;
    }
    const uint32_t nwords = 4u * ((tot + 127u) / 128u);
    const uint32_t grp = it.c >> GRP_SHIFT;
    if (tid == 0) {                                   // publish this chunk's size
        *reinterpret_cast<volatile uint32_t*>(p.enc_st + item) = ST_VALID | nwords;
        atomicAdd(p.enc_grp + (size_t)it.u * p.n_grp + grp,
                  (1ull << 56) | ((unsigned long long)nwords << 32) | (unsigned long long)tot);
    }
    for (uint32_t i = tid; i < nwords / 4 + 1; i += ENC_THREADS) reinterpret_cast<uint4*>(s_buf)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < RUNS_PER_THREAD; ++k) {
        if (mask[k] == 0u) continue;
        uint32_t at = pos[k];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            put_piece(s_buf, at, piece[k][q]);
            at += (plen[k] >> (8 * q)) & 0xFFu;
        }
    }
    // offset of the chunk = words of all earlier chunks of this user
    bool timeout = false;
    uint32_t sum = 0;
    for (uint32_t i = tid; i < grp; i += ENC_THREADS)
        sum += (uint32_t)(wait_group(p.enc_grp + (size_t)it.u * p.n_grp + i, GRP_SIZE, p.spin_limit, timeout) >> 32);
    if ((uint32_t)tid < (it.c & (GRP_SIZE - 1)))
        sum += wait_count(p.enc_st + (size_t)it.u * p.n_chunks + ((size_t)grp << GRP_SHIFT) + tid, p.spin_limit, timeout);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) s_sum[warp] = sum;
    const int any_timeout = __syncthreads_or(timeout);                // also: the image is complete
    uint32_t dst_word = 0;
#pragma unroll
    for (int w = 0; w < ENC_WARPS; ++w) dst_word += s_sum[w];
    if (tid == 0) {
        uint32_t* co = chunk_off + (size_t)it.u * (p.n_chunks + 1);
        co[it.c] = dst_word;
        if ((int64_t)it.c == p.n_chunks - 1) co[p.n_chunks] = dst_word + nwords;
        if (bad) atomicOr(p.flags, CO3_FLAG_CORRUPT);
        if (any_timeout) atomicOr(p.flags, CO3_FLAG_TIMEOUT);
        if ((int64_t)dst_word + nwords > p.cap_words) atomicOr(p.flags, CO3_FLAG_CAPACITY);
    }
    if ((int64_t)it.c == p.n_chunks - 1 && warp == 0) {
        // the user's last chunk: every chunk of the user has a smaller ticket, so all groups fill up;
        // r_t^(u) = code bits of the user = sum of the groups' bit totals
        bool t2 = false;
        unsigned long long ub = 0;
        for (uint32_t i = lane; i <= grp; i += 32) {
            const uint32_t expect = (i < grp) ? (uint32_t)GRP_SIZE : (it.c & (GRP_SIZE - 1)) + 1u;
            ub += wait_group(p.enc_grp + (size_t)it.u * p.n_grp + i, expect, p.spin_limit, t2) & 0xFFFFFFFFull;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ub += __shfl_xor_sync(0xffffffffu, ub, o);
        if (lane == 0) user_bits[it.u] = ub;
        if (t2 && lane == 0) atomicOr(p.flags, CO3_FLAG_TIMEOUT);
    }
    if (any_timeout || (int64_t)dst_word + nwords > p.cap_words) return;   // nothing is written outside the row
    uint4* dst = reinterpret_cast<uint4*>(bitstream + (size_t)it.u * p.cap_words + dst_word);
    const uint4* srcv = reinterpret_cast<const uint4*>(s_buf);
    for (uint32_t i = tid; i < nwords / 4; i += ENC_THREADS) dst[i] = srcv[i];
}

// Fully lagged code: the convert-and-pack pass left every sub-chunk packed from bit 0 of its own
// staging slot.  One block per chunk shifts the sub-chunks to their places in a shared image of the
// chunk (a scan of their bit counts) and stores the image at the chunk's place in the payload.
constexpr int CAT_THREADS = 64;
__global__ void __launch_bounds__(CAT_THREADS)
enc_concat_kernel(Co3Dev p, const uint16_t* __restrict__ sub_bits, const uint32_t* __restrict__ chunk_off,
                  uint32_t* __restrict__ bitstream) {
    __shared__ __align__(16) uint32_t s_img[BUF_WORDS + 4];
    __shared__ uint32_t s_pos[CO3_TILE / CO3_SUB], s_nb[CO3_TILE / CO3_SUB];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t item = blockIdx.x;
    const uint32_t n_chunks = (uint32_t)p.n_chunks;
    const uint32_t u = item / n_chunks, c = item - u * n_chunks;
    // every load that does not depend on another one is issued here, before any is used
    const uint32_t* stage = p.slot_buf + (size_t)item * CO3_SLOT_WORDS;
    constexpr int PER_WARP = (CO3_TILE / CO3_SUB) / (CAT_THREADS / 32);     // sub-chunks per warp (4)
    uint32_t v[PER_WARP];
#pragma unroll
    for (int k = 0; k < PER_WARP; ++k)                // first 32 words of each slot (what 8 bits per symbol fill)
        v[k] = __ldg(stage + (warp + (CAT_THREADS / 32) * k) * CO3_SUB_WORDS + lane);
    const uint32_t ovf = p.user_ovf[u];
    const uint32_t nwords = p.chunk_words[item];
    const uint32_t dst_word = chunk_off[(size_t)u * (p.n_chunks + 1) + c];
    const Co3Chunk cd = p.chunks[c];
    if (ovf) return;                                  // this user's payload does not fit: row left untouched
    const int tlo = (int)(cd.start & (CO3_TILE - 1));
    const int sub_first = tlo / CO3_SUB, sub_last = (tlo + cd.len - 1) / CO3_SUB;
    if (warp == 0) {                                  // lane = sub-chunk of the tile
        const bool in = lane >= sub_first && lane <= sub_last;
        const uint32_t nb = in ? sub_bits[(size_t)u * p.n_sub + cd.sub0 + (lane - sub_first)] : 0u;
        uint32_t x = nb;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        s_pos[lane] = x - nb;
        s_nb[lane] = nb;
    }
    for (uint32_t i = tid; i < nwords / 4 + 1; i += CAT_THREADS) reinterpret_cast<uint4*>(s_img)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < PER_WARP; ++k) {
        const int sc = warp + (CAT_THREADS / 32) * k;
        const uint32_t pos = s_pos[sc], nb = s_nb[sc];
        if (32u * lane < nb) {
            const uint32_t at = pos + 32u * lane, wi = at >> 5, sh = at & 31u;
            atomicOr(&s_img[wi], v[k] << sh);
            if (sh) atomicOr(&s_img[wi + 1], v[k] >> (32u - sh));
        }
        const uint32_t i = lane + 32;                 // second half: only above 8 bits per symbol
        if (32u * i < nb) {
            const uint32_t w = stage[sc * CO3_SUB_WORDS + i];
            const uint32_t at = pos + 32u * i, wi = at >> 5, sh = at & 31u;
            atomicOr(&s_img[wi], w << sh);
            if (sh) atomicOr(&s_img[wi + 1], w >> (32u - sh));
        }
    }
    __syncthreads();
    uint4* dst = reinterpret_cast<uint4*>(bitstream + (size_t)u * p.cap_words + dst_word);
    const uint4* srcv = reinterpret_cast<const uint4*>(s_img);
    for (uint32_t i = tid; i < nwords / 4; i += CAT_THREADS) dst[i] = srcv[i];
}

}  // namespace

// 64 threads per chunk (four runs each, 72 registers, 14 blocks per SM).  Measured against it on the
// 8-user ResNet-18 workload: 128 threads with two runs each (48 registers, 40 warps per SM) is 6 % slower
// (twice the per-thread fixed work and four warps at every barrier), 12 or 16 blocks per SM within 2 %.
static void launch_enc_single(const Co3Dev& p, const co3_seg_header* hdr, uint16_t* sub_bits, uint32_t* chunk_off,
                              unsigned long long* user_bits, uint32_t* bitstream, unsigned blocks, unsigned items,
                              cudaStream_t st) {
    enc_single_kernel<64, 14><<<blocks, 64, 0, st>>>(p, hdr, sub_bits, chunk_off, user_bits, bitstream, items);
}

cudaError_t co3_setup_kernels(void) { return cudaSuccess; }

cudaError_t co3_launch_scan_gather(co3_plan* pl, uint32_t* bitstream, const uint16_t* sub_bits, uint32_t* chunk_off,
                                   unsigned long long* user_bits, cudaStream_t st) {
    const Co3Dev& p = pl->dev;
    const unsigned items = (unsigned)(p.n_chunks * (int64_t)p.U);
    cudaError_t e;
    co3_prof_begin(pl, CO3_K_ENC_SCAN, st);
    enc_scan_kernel<<<p.U, 1024, 0, st>>>(p, chunk_off, user_bits);
    co3_prof_end(pl, CO3_K_ENC_SCAN, st, 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    co3_prof_begin(pl, CO3_K_ENC_PACK, st);
    enc_concat_kernel<<<items, CAT_THREADS, 0, st>>>(p, sub_bits, chunk_off, bitstream);
    co3_prof_end(pl, CO3_K_ENC_PACK, st, 1);
    return cudaGetLastError();
}

cudaError_t co3_launch_encode(co3_plan* pl, const co3_seg_header* hdr, uint32_t* bitstream,
                              uint16_t* sub_bits, uint32_t* chunk_off, unsigned long long* user_bits,
                              cudaStream_t st) {
    Co3Dev p = pl->dev;
    if (pl->cfg.bias_mode == CO3_CODE_EMPIRICAL) { p.cb = pl->cb_emp; p.code_by_segment = 1; }
    const unsigned items = (unsigned)(p.n_chunks * (int64_t)p.U);
    // (tickets, published counts and group totals were cleared by the fit kernel that ran before)
    co3_prof_begin(pl, CO3_K_ENC_PACK, st);
    launch_enc_single(p, hdr, sub_bits, chunk_off, user_bits, bitstream, items, items, st);
    co3_prof_end(pl, CO3_K_ENC_PACK, st, 1);
    return cudaGetLastError();
}

// Test hook behind co3_debug_encode_stalled: the same kernel over the symbols of the last iteration,
// but the tickets start at 1 and one block fewer is launched, so item 0 (user 0, chunk 0) is never
// claimed and never publishes its size.  Every block that needs that size polls spin_limit times, gives
// up, raises CO3_FLAG_TIMEOUT and writes no payload; nothing waits without a limit.
cudaError_t co3_launch_encode_stalled(co3_plan* pl, const co3_seg_header* hdr, uint32_t* bitstream,
                                      uint16_t* sub_bits, uint32_t* chunk_off, unsigned long long* user_bits,
                                      int spin_limit, cudaStream_t st) {
    Co3Dev p = pl->dev;
    const unsigned items = (unsigned)(p.n_chunks * (int64_t)p.U);
    if (items < 2) return cudaErrorInvalidValue;
    p.spin_limit = spin_limit;
    cudaError_t e = cudaMemsetAsync(p.enc_grp, 0, pl->enc_sync_bytes, st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(p.enc_ticket, 1, 1, st);       // low byte of the zeroed ticket: the first ticket drawn is 1
    if (e != cudaSuccess) return e;
    launch_enc_single(p, hdr, sub_bits, chunk_off, user_bits, bitstream, items - 1, items, st);
    pl->launches += 1;
    return cudaGetLastError();
}
