// Parameter-server side (Algorithm 1 lines 13-14 up to the model update, Eq. "aggregate"):
// decode every user's stream and write the average of the reconstructed gradients.
//
// A lane decodes one sub-chunk (<= 128 codewords) serially with a primary table (13 or 11 index bits)
// whose entries already hold the signed integer magnitude ((K << 8) | length) -- longer codewords
// go through a second table in global memory; the 32 sub-chunks of a
// chunk are the 32 lanes of a warp, so a warp is one (chunk, user) stream.  The magnitudes of all
// users are accumulated with shared-memory reductions into a transposed, padded tile
// (conflict-free both for the per-lane scattered adds and for the coalesced read-out), scaled
// once by 2^lambda and divided by U.  The stream words are staged in shared memory with 128-bit
// loads, so global traffic is fully coalesced.
//
// The inner loop is written for issue slots: shared memory is addressed with 32-bit
// shared-space addresses (ld.shared / red.shared), the funnel shifts take the table entry itself
// as shift amount (only its low five bits count), the bit buffer is topped up once per pair of
// symbols, and four symbols are decoded per loop trip with immediate accumulator offsets.
//
// Three kernels.  U = 1 has nothing to add up: 24 independent warps per block, each transposing its
// own stream through a small tile.  2 <= U <= 8 keeps one stream per warp and walks the chunk in quarters of 32 symbols
// per sub-chunk (small double-buffered accumulator, several chunks per group when U < 8); the
// whole table entries are accumulated (the length bytes of at most 8 users cannot carry into
// the magnitude) and the magnitude sum is taken out with one shift at the end.  U > 8 keeps a
// whole-chunk accumulator and loops over the users.
// Both run several 8-warp teams in one block per SM (1024 threads for U = 8 and U > 8): the teams
// share one table of 13 or 12 index bits (with 11 bits one group of 128 look-ups in eight still meets
// a longer codeword and leaves the fast path, which also makes the warps of a team wait for each
// other), each team has its own named barrier, and the whole block synchronises only where the
// segment (the table) changes.  User counts that do not divide 8 keep one-team blocks, four per SM,
// with an 11-bit table.
//
// Bound: HBM for U = 1 (4 B written per element); for U >= 4 the serial decode (issue slots and
// shared-memory wavefronts: the table look-up of 32 lanes hits random banks) dominates.
#include "co3_internal.h"

namespace {

constexpr int NW = CO3_THREADS / 32;              // warps = concurrent streams per block
constexpr int PADW = 33;                          // row stride of the transposed accumulator
// A lane never reads more than 128 * 16 bits (plus the three words its reader holds ahead) past the
// start of its sub-chunk, so with this much slack after the staged words the staged reader needs no
// bounds checks.
constexpr int STAGE_PAD = 72;
constexpr int STAGE_ROW = CO3_STAGE_WORDS + STAGE_PAD;
static_assert(STAGE_ROW % 4 == 0, "stage rows must keep 16-byte alignment");

// The long codewords of a good code carry about as much Kraft mass as probability (~1e-3 of 65536
// windows), so the head of the second table that fits here nearly always holds all of them.
constexpr int LONG_CACHE = CO3_LONG_CACHE;

// (The primary table itself is a static __shared__ array of each kernel, so that its address is a
// constant of the load instruction and a look-up is mask, load; `lut` points to it for the rare paths.)
template <int BITS>
struct TablesT {                                  // per-segment decoder tables in shared memory
    static constexpr int bits = BITS;
    static_assert(BITS <= 14, "two codewords of the primary table must fit the 30 bits a refill guarantees");
    uint32_t* lut;
    alignas(16) uint32_t long_cache[LONG_CACHE];  // the row's second table from the first codeword longer than BITS
    const uint32_t* lut_long;                     // the rest of it (global memory)
    uint32_t long_first;                          // first 16-bit window it covers
    uint32_t long_n;                              // number of windows it covers
};

__device__ __forceinline__ uint32_t keep_up_to(uint32_t e, uint32_t bits) { return (e & 0xFFu) > bits ? 0u : e; }

// The stored table has 2^13 entries indexed by the next 13 stream bits (first bit lowest); its first
// 2^BITS entries are the table for BITS index bits once the entries of longer codewords are blanked.
template <int BITS>
__device__ void load_tables(TablesT<BITS>& t, uint32_t* s_lut, const Co3CodeBook& cb, int row, int tid, int nthreads) {
    const uint4* lut = reinterpret_cast<const uint4*>(cb.lut + (size_t)row * CO3_LUT_SIZE);
    uint4* dst = reinterpret_cast<uint4*>(s_lut);
    if (tid == 0) t.lut = s_lut;
    for (int i = tid; i < (1 << BITS) / 4; i += nthreads) {
        uint4 v = __ldg(lut + i);
        if (BITS < CO3_LUT_BITS) {
            v.x = keep_up_to(v.x, BITS); v.y = keep_up_to(v.y, BITS);
            v.z = keep_up_to(v.z, BITS); v.w = keep_up_to(v.w, BITS);
        }
        dst[i] = v;
    }
    // the second table starts at the first window of a 12-bit codeword; this decoder enters it at the
    // first window of a codeword longer than BITS (both multiples of 4, so are the row lengths)
    const uint32_t* first = cb.first + (size_t)row * (CO3_MAXLEN + 1);
    const uint32_t tab_first = __ldg(first + CO3_LONG_FROM) << (CO3_MAXLEN - CO3_LONG_FROM);
    const uint32_t my_first = BITS + 1 == CO3_LONG_FROM ? tab_first : __ldg(first + BITS + 1) << (CO3_MAXLEN - BITS - 1);
    const uint32_t base = my_first - tab_first, stride = (uint32_t)cb.long_stride;
    const uint32_t* lg = cb.lut_long + (size_t)row * cb.long_stride;
    if (tid < LONG_CACHE / 4) {
        const uint32_t i = base + 4u * (uint32_t)tid;
        reinterpret_cast<uint4*>(t.long_cache)[tid] =
            i + 3u < stride ? __ldg(reinterpret_cast<const uint4*>(lg + i)) : make_uint4(0, 0, 0, 0);
    }
    if (tid == 0) {
        t.lut_long = lg + (base < stride ? base : 0u);
        t.long_first = my_first;
        t.long_n = base < stride ? stride - base : 0u;
    }
}

__device__ __forceinline__ float pow2_clamped(int e) {   // 2^e; a corrupt header cannot make a NaN
    e = min(max(e, -126), 127);
    return __uint_as_float((uint32_t)(e + 127) << 23);
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
template <int OFF>
__device__ __forceinline__ void red_add(uint32_t addr, uint32_t v) {
    asm volatile("red.shared.add.u32 [%0+%2], %1;" ::"r"(addr), "r"(v), "n"(OFF) : "memory");
}

// Codeword longer than the primary table: one look-up in the row's second table (its head is in
// shared memory, the rest in global memory; about one symbol in a thousand comes here).  Returns the entry (K << 8) | length.
template <class T>
__device__ __forceinline__ uint32_t decode_long(uint32_t window, const T& t, bool& bad) {
    const uint32_t v = __brev(window) >> 16;      // 16 stream bits, root bit on top
    const uint32_t i = v - t.long_first;
    uint32_t e = i < LONG_CACHE ? t.long_cache[i] : (i < t.long_n ? __ldg(t.lut_long + i) : 0u);
    if ((e & 0xFFu) == 0u) {                      // no codeword starts like this: corrupt stream
        bad = true;
        e = CO3_MAXLEN;
    }
    return e;
}

// LSB-first bit reader over staged words.  The window hi:lo holds the stream SHIFTED LEFT BY TWO: the
// next stream bits sit at bits [2, nb) and the bits above are zero, so that `lo & (mask << 2)` is at
// once the byte offset of the table entry (bits 0 and 1 hold leftovers of consumed codewords, which
// the mask drops).  nb therefore counts the stream bits in the window plus two.  nw is the word after
// those, already loaded (a refill takes it and loads the one after, so that no refill waits for
// shared memory), and rp the shared-space byte address of the word after nw.  A refill is checked once
// per PAIR of symbols: with nb >= 32 the window holds at least 30 stream bits, which two codewords of
// the primary table (at most 14 bits each) or one of any length (16) never exceed, and with nb < 32
// one more word always fits.  (With 32 lanes a per-symbol refill branch would be taken on nearly every
// step, so its cost is paid per step, not per refill.)
// nb is kept in the low byte of its register only: a step subtracts the whole table entry (length in
// the low byte, which never borrows because nb >= length + 2), and the shifts look at five bits (a
// refill finds 2 <= nb <= 31).
struct Reader {
    uint32_t lo, hi;
    uint32_t nb;
    uint32_t rp;
    uint32_t nw;                                  // the word before rp: fetched one refill before it is used
};

__device__ __forceinline__ uint32_t reader_bits(const Reader& r) { return r.nb & 0xFFu; }

__device__ __forceinline__ void refill(Reader& r) {
    if (reader_bits(r) < 32u) {                               // then hi holds no bit
        const uint32_t w = r.nw;
        r.nw = lds32(r.rp);                                   // not needed before the next refill
        r.lo |= __funnelshift_l(0u, w, r.nb);                 // w << nb
        r.hi = __funnelshift_l(w, 0u, r.nb);                  // w >> (32 - nb)
        r.nb += 32u;
        r.rp += 4;
    }
}

__device__ __forceinline__ void reader_init(Reader& r, uint32_t stage_addr, uint32_t bitpos) {
    r.rp = stage_addr + ((bitpos >> 5) << 2);
    const uint32_t sh = bitpos & 31u;
    const uint32_t w0 = lds32(r.rp) >> sh;                    // the 32 - sh bits left of the first word
    r.lo = w0 << 2;
    r.hi = w0 >> 30;
    r.nb = 34u - sh;
    r.nw = lds32(r.rp + 4);
    r.rp += 8;
}
// stream bits consumed since bit 0 of the staged words
__device__ __forceinline__ uint32_t reader_pos(const Reader& r, uint32_t stage_addr) {
    return ((r.rp - stage_addr - 4u) << 3) + 2u - reader_bits(r);
}
// the next 30 stream bits, unshifted (for the second table)
__device__ __forceinline__ uint32_t reader_window(const Reader& r) { return __funnelshift_r(r.lo, r.hi, 2); }

template <int OFF>
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u32 [%0+%2], %1;" ::"r"(addr), "r"(v), "n"(OFF) : "memory");
}
// What a decoded symbol does to its cell: added (several users meet there) or stored (one user: the
// cell is this lane's alone and holds the whole table entry until the read-out).
template <int OFF, bool STORE>
__device__ __forceinline__ void put_cell(uint32_t addr, uint32_t v) {
    if (STORE) sts32<OFF>(addr, v);
    else red_add<OFF>(addr, v);
}

// One symbol, fast form: look up, consume, add to the accumulator row at byte offset OFF, return
// the table entry.  No test for a codeword longer than the table: such an entry is 0 (nothing is
// consumed, nothing is added), so every later look-up of the group sees the same window and returns 0
// too, and the caller tests only the group's LAST entry.
// PACKED: add the whole entry (length byte included); else add the signed magnitude.
template <int OFF, bool PACKED, int BITS, bool STORE = false>
__device__ __forceinline__ uint32_t decode_step(Reader& r, const unsigned char* lut, uint32_t acc_addr) {
    const uint32_t e = *reinterpret_cast<const uint32_t*>(lut + (r.lo & (((1u << BITS) - 1u) << 2)));
    r.lo = __funnelshift_r(r.lo, r.hi, e);        // shift by the length: low five bits of e
    r.hi = __funnelshift_r(r.hi, 0u, e);
    r.nb -= e;                                    // the low byte counts
    put_cell<OFF, STORE>(acc_addr, PACKED ? e : (uint32_t)((int32_t)e >> 8));
    return e;
}

// One symbol with the test for a long codeword (group tails, and groups that met a long codeword).
template <bool PACKED, class T, bool STORE = false>
__device__ __forceinline__ void decode_step_checked(Reader& r, const unsigned char* lut, uint32_t acc_addr,
                                                    const T& t, bool& bad) {
    uint32_t e = *reinterpret_cast<const uint32_t*>(lut + (r.lo & (((1u << T::bits) - 1u) << 2)));
    if ((e & 0xFFu) == 0u) e = decode_long(reader_window(r), t, bad);
    r.lo = __funnelshift_r(r.lo, r.hi, e);
    r.hi = __funnelshift_r(r.hi, 0u, e);
    r.nb -= e;                                    // the low byte counts
    put_cell<0, STORE>(acc_addr, PACKED ? e : (uint32_t)((int32_t)e >> 8));
}

// A group of four whose fast pass stopped at a long codeword after `done` good symbols: the reader
// stands exactly at that codeword, so the rest of the group is decoded with the checked step.
// Rare (about one symbol in a thousand is longer than the table).  Inlined, so that the reader stays
// in registers (its address is never taken); the long-codeword search itself is out of line.
// (ROW: words between the cells of consecutive symbols of a lane)
template <bool PACKED, class T, bool STORE = false, int ROW = PADW>
__device__ __forceinline__ void finish_group(Reader& r, const unsigned char* lut_addr, uint32_t acc_addr, int done,
                                             const T& t, bool& bad) {
#pragma unroll 1
    for (int k = done; k < 4; ++k) {
        refill(r);
        decode_step_checked<PACKED, T, STORE>(r, lut_addr, acc_addr + (uint32_t)k * (ROW * 4), t, bad);
    }
}

template <bool PACKED, class T, bool STORE = false, int ROW = PADW>
__device__ __forceinline__ void decode_run(Reader& r, const unsigned char* lut_addr, uint32_t acc_addr, int n,
                                           const T& t, bool& bad) {
    int i = 0;
    for (; i + 4 <= n; i += 4) {
        refill(r);
        const uint32_t e0 = decode_step<0, PACKED, T::bits, STORE>(r, lut_addr, acc_addr);
        const uint32_t e1 = decode_step<ROW * 4, PACKED, T::bits, STORE>(r, lut_addr, acc_addr);
        refill(r);
        const uint32_t e2 = decode_step<ROW * 8, PACKED, T::bits, STORE>(r, lut_addr, acc_addr);
        const uint32_t e3 = decode_step<ROW * 12, PACKED, T::bits, STORE>(r, lut_addr, acc_addr);
        if ((e3 & 0xFFu) == 0u) {
            const int done = ((e0 & 0xFFu) != 0u) + ((e1 & 0xFFu) != 0u) + ((e2 & 0xFFu) != 0u);
            finish_group<PACKED, T, STORE, ROW>(r, lut_addr, acc_addr, done, t, bad);
        }
        acc_addr += ROW * 16;
    }
    for (; i < n; ++i) {
        refill(r);
        decode_step_checked<PACKED, T, STORE>(r, lut_addr, acc_addr, t, bad);
        acc_addr += ROW * 4;
    }
}

// The same for a stream that did not fit the staging row: words come from global memory with
// bounds checks.  Rare (a chunk above 8 bits per symbol), so written plainly.
struct SlowReader {
    unsigned long long buf;
    int nb;
    uint32_t wp;
};
__device__ __forceinline__ uint32_t fetch_checked(const uint32_t* src, uint32_t nwords, uint32_t i) {
    return i < nwords ? src[i] : 0u;
}
__device__ void slow_init(SlowReader& r, const uint32_t* src, uint32_t nwords, uint32_t bitpos) {
    r.wp = bitpos >> 5;
    const uint32_t sh = bitpos & 31u;
    r.buf = (unsigned long long)(fetch_checked(src, nwords, r.wp) >> sh);
    r.nb = 32 - (int)sh;
    r.wp++;
    r.buf |= (unsigned long long)fetch_checked(src, nwords, r.wp) << r.nb;
    r.nb += 32;
    r.wp++;
}
template <bool PACKED, class T, bool STORE = false, int ROW = PADW>
__device__ void slow_run(SlowReader& r, const T& t, const uint32_t* src, uint32_t nwords, int32_t* acc,
                         int n, bool& bad) {
    for (int i = 0; i < n; ++i) {
        const uint32_t window = (uint32_t)r.buf;
        uint32_t e = t.lut[window & ((1u << T::bits) - 1u)];
        if ((e & 0xFFu) == 0u) e = decode_long(window, t, bad);
        const uint32_t len = e & 0xFFu;
        r.buf >>= len;
        r.nb -= (int)len;
        if (STORE) *acc = PACKED ? (int32_t)e : ((int32_t)e >> 8);
        else atomicAdd(acc, PACKED ? (int32_t)e : ((int32_t)e >> 8));
        acc += ROW;
        if (r.nb < 32) {
            r.buf |= (unsigned long long)fetch_checked(src, nwords, r.wp) << r.nb;
            r.nb += 32;
            r.wp++;
        }
    }
}

struct Stream {                                   // one (chunk, user) stream as seen by a lane
    uint32_t nwords;
    uint32_t bitpos;                              // start of this lane's sub-chunk
    uint32_t sub_len_bits;                        // recorded length of this lane's sub-chunk
    int i_lo, i_hi;                               // this lane's symbols within its 128-window
    bool active;
    bool staged;                                  // words are in shared memory (else read from global)
    const uint32_t* gsrc;
};

// Stage the words of (chunk c, user u) into `stage` (if they fit) and give every lane the start
// of its sub-chunk.  Called by one whole warp.
__device__ __forceinline__ void open_stream(Stream& s, const Co3Dev& p, const Co3Chunk& cd, int64_t c, int u,
                                            const uint32_t* __restrict__ bitstream,
                                            const uint16_t* __restrict__ sub_bits,
                                            uint32_t w0, uint32_t w1,      // chunk_off[u][c], chunk_off[u][c + 1]
                                            uint32_t* stage, int lane, bool& bad) {
    uint32_t nwords = 0;
    if ((w0 & 3u) || w1 < w0 || (int64_t)w1 > p.cap_words) bad = true;   // offsets must be sane
    else nwords = w1 - w0;
    const uint32_t* g = bitstream + (size_t)u * p.cap_words + (nwords ? w0 : 0u);
    s.gsrc = g;
    s.staged = nwords <= CO3_STAGE_WORDS;
    if (s.staged) {
        // asynchronous 16-byte copies: all of a lane's (up to eight) are in flight together, and the
        // side information below is fetched while they are; waited for at the end
        const uint32_t sdst = (uint32_t)__cvta_generic_to_shared(stage);
        for (uint32_t i = lane; i < nwords / 4; i += 32)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(sdst + 16u * i), "l"(g + 4u * i) : "memory");
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    }
    s.nwords = nwords;
    const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
    const int lo = (int)(cd.start - tb), hi = lo + cd.len;
    const int sub_first = lo / CO3_SUB, sub_last = (hi - 1) / CO3_SUB;
    s.active = lane >= sub_first && lane <= sub_last;
    s.i_lo = max(lo - lane * CO3_SUB, 0);
    s.i_hi = min(hi - lane * CO3_SUB, CO3_SUB);
    uint32_t sb = s.active ? sub_bits[(size_t)u * p.n_sub + cd.sub0 + (lane - sub_first)] : 0u;
    uint32_t x = sb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    s.bitpos = x - sb;
    s.sub_len_bits = sb;
    if (s.bitpos > nwords * 32u) {                // a start outside the chunk: corrupt side info
        bad = true;
        s.bitpos = nwords * 32u;
    }
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncwarp();
}

// Algorithm 1 line 14, optional: w <- w + step * avg (two roundings; the caller chooses the sign).
__device__ __forceinline__ void put_out(float* avg, float* weights, float step, int64_t i, float v) {
    avg[i] = v;
    if (weights) weights[i] = __fadd_rn(weights[i], __fmul_rn(step, v));
}

__device__ __forceinline__ float finish(int32_t ksum, float scale, float fu, float inv_u) {
    const float v = __fmul_rn((float)ksum, scale);                  // exact
    return inv_u != 0.0f ? __fmul_rn(v, inv_u) : __fdiv_rn(v, fu);  // U a power of two: exact either way
}

// ---- U <= 8: one stream per warp, quarter batches ------------------------------------------
// A team = 8 warps = NW / U chunks x U users.  TEAMS teams share the block's tables (BITS index
// bits: as wide as the shared memory left by the teams allows); a team has its own named barrier,
// and the block synchronises as a whole only where the segment (the table) changes.
constexpr int QB = 32;                            // symbols per lane per batch
// descriptors a block keeps in shared memory (the rest: global), as many as the variant has room for
__host__ __device__ constexpr int desc_chunks(int UC) { return UC == NW ? 128 : 48; }
__host__ __device__ constexpr size_t desc_bytes(int UC) {
    return desc_chunks(UC) * (sizeof(Co3Group) + sizeof(Co3Chunk));
}
constexpr int ACC_Q = QB * PADW;                  // accumulator words per chunk per batch

struct TeamHead {                                 // followed by the accumulator: [2][chunks per group][ACC_Q]
    long long c_tb[2][NW];                        // per chunk of the group: tile base, bounds in the tile
    int c_lo[2][NW], c_hi[2][NW];                 // (two sets: a group is read out while the next one opens)
    alignas(16) uint32_t stage[NW][STAGE_ROW];    // filled with 128-bit stores
};
static_assert(sizeof(TeamHead) % 16 == 0, "the accumulator behind it is cleared with 128-bit stores");

__host__ __device__ inline int acc_words_a(int U) { return ((NW / U) * ACC_Q + 3) & ~3; }
__host__ __device__ inline size_t team_bytes(int U) { return sizeof(TeamHead) + sizeof(int32_t) * 2 * (size_t)acc_words_a(U); }
template <int TEAMS, int BITS>
__host__ __device__ inline size_t smem_a_bytes(int U) { return sizeof(TablesT<BITS>) + TEAMS * team_bytes(U); }

__device__ __forceinline__ void team_barrier(int team) {   // barrier 0 is the block's own
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "n"(CO3_THREADS) : "memory");
}

// One quarter of one chunk: scale the sums of warp w's sub-chunks (w, w + 8, ...) and zero them.
__device__ __forceinline__ void read_out(int32_t* a, int64_t o, int e0, int lo, int hi, float scale, float fu,
                                         float inv_u, float* avg, float* weights, float step) {
    if (lo == 0 && hi == CO3_TILE) {
#pragma unroll
        for (int rr = 0; rr < 32 * QB / CO3_THREADS; ++rr) {
            put_out(avg, weights, step, o + rr * NW * CO3_SUB, finish(a[rr * NW] >> 8, scale, fu, inv_u));
            a[rr * NW] = 0;
        }
    } else {
#pragma unroll
        for (int rr = 0; rr < 32 * QB / CO3_THREADS; ++rr) {
            const int e = e0 + rr * NW * CO3_SUB;
            if (e >= lo && e < hi) put_out(avg, weights, step, o + rr * NW * CO3_SUB, finish(a[rr * NW] >> 8, scale, fu, inv_u));
            a[rr * NW] = 0;
        }
    }
}

// UC: the number of users when it is known at compile time (the powers of two), else 0.
template <int TEAMS, int BITS, int UC>
__global__ void __launch_bounds__(TEAMS * CO3_THREADS, TEAMS == 1 ? 4 : 1)
decode_small_u_kernel(Co3Dev p, const uint32_t* __restrict__ bitstream,
                      const uint16_t* __restrict__ sub_bits, const uint32_t* __restrict__ chunk_off,
                      const co3_seg_header* __restrict__ hdr, float* __restrict__ avg,
                      float* __restrict__ weights, float step) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    TablesT<BITS>& tabs = *reinterpret_cast<TablesT<BITS>*>(s_raw);
    const int tid = threadIdx.x, lane = tid & 31;
    const int team = tid / CO3_THREADS, ttid = tid - team * CO3_THREADS, warp = ttid >> 5;
    const int U = UC ? UC : p.U;
    const bool all_mine = UC == NW;                // one chunk per group and every warp has a stream of it
    unsigned char* team_raw = s_raw + sizeof(TablesT<BITS>) + (size_t)team * team_bytes(U);
    TeamHead& tm = *reinterpret_cast<TeamHead*>(team_raw);
    int32_t* acc0 = reinterpret_cast<int32_t*>(team_raw + sizeof(TeamHead));
    const int cpg = NW / U;                        // chunks per group (>= 1)
    const int accw = acc_words_a(U);               // words per accumulator buffer
    __shared__ __align__(16) uint32_t s_lut[1 << BITS];
    const unsigned char* lut_addr = reinterpret_cast<const unsigned char*>(s_lut);
    const uint32_t acc_addr0 = (uint32_t)__cvta_generic_to_shared(acc0);
    const uint32_t stage_addr = (uint32_t)__cvta_generic_to_shared(tm.stage[warp]);
    const int ci = warp / U, us = warp - ci * U;   // this warp's chunk-in-group and user
    const int64_t g0 = p.dec_part[blockIdx.x], g1 = p.dec_part[blockIdx.x + 1];
    const float fu = (float)U;
    const float inv_u = (U & (U - 1)) == 0 ? 1.0f / fu : 0.0f;
    bool bad = false;
    // The descriptors of the block's first groups and chunks go to shared memory: a stream's side
    // information is addressed through them, and fetched from global memory they are a dependent load in
    // front of every stream.
    constexpr int DESC_CHUNKS = desc_chunks(UC), DESC_GROUPS = DESC_CHUNKS;
    __shared__ Co3Group s_grp[DESC_GROUPS];
    __shared__ Co3Chunk s_chk[DESC_CHUNKS];
    const int64_t chunk_base = g0 < g1 ? p.groups[g0].chunk0 : 0;
    for (int64_t i = tid; i < min(g1 - g0, (int64_t)DESC_GROUPS); i += TEAMS * CO3_THREADS) s_grp[i] = p.groups[g0 + i];
    for (int64_t i = tid; i < DESC_CHUNKS && chunk_base + i < p.n_chunks; i += TEAMS * CO3_THREADS) s_chk[i] = p.chunks[chunk_base + i];
    auto group_of = [&](int64_t g) { return g - g0 < DESC_GROUPS ? s_grp[g - g0] : p.groups[g]; };
    auto chunk_of = [&](int64_t c) { return c - chunk_base < DESC_CHUNKS ? s_chk[c - chunk_base] : p.chunks[c]; };
    int opened = 0;                                // groups this team has opened
    // Both accumulator buffers start at zero and every read-out zeroes what it has read, so one
    // barrier per quarter is enough: decode(q) -> barrier -> read-out(q), and the buffer of quarter q
    // is next written after the barrier of quarter q + 1.
    for (int i = ttid; i < 2 * accw / 4; i += CO3_THREADS) reinterpret_cast<uint4*>(acc0)[i] = make_uint4(0, 0, 0, 0);
    int64_t gi = g0;
    while (gi < g1) {                              // one trip per run of groups of one segment
        const int seg = p.groups[gi].seg;
        int64_t ge = gi + 1;
        while (ge < g1 && p.groups[ge].seg == seg) ++ge;
        __syncthreads();                           // every team is past its last look-up in the old tables
        load_tables(tabs, s_lut, p.cb, p.code_by_segment ? seg : co3_row_of(hdr[seg], &bad), tid, TEAMS * CO3_THREADS);
        __syncthreads();                           // (and the first zeroing)
        const float scale = pow2_clamped((int)hdr[seg].bias + p.cF);
        for (int64_t g = gi + team; g < ge; g += TEAMS, ++opened) {
            const Co3Group grp = group_of(g);
            const int gp = opened & 1;
            const bool mine = all_mine || (ci < cpg && ci < grp.count);
            Stream s;
            s.active = false; s.staged = true; s.nwords = 0; s.bitpos = 0; s.sub_len_bits = 0;
            s.i_lo = 0; s.i_hi = 0; s.gsrc = nullptr;
            Reader r;
            r.lo = 0; r.hi = 0; r.nb = 0; r.rp = stage_addr; r.nw = 0;
            SlowReader sr;
            sr.buf = 0; sr.nb = 0; sr.wp = 0;
            long long my_tb = 0;                   // bounds of this warp's own chunk (used when all_mine)
            int my_lo = 0, my_hi = 0;
            if (mine) {
                const Co3Chunk cd = chunk_of(grp.chunk0 + ci);
                const int64_t cc = grp.chunk0 + ci;
                const uint32_t* co = chunk_off + (size_t)us * (p.n_chunks + 1) + cc;
                open_stream(s, p, cd, cc, us, bitstream, sub_bits, co[0], co[1], tm.stage[warp], lane, bad);
                if (s.active) {
                    if (s.staged) reader_init(r, stage_addr, s.bitpos);
                    else slow_init(sr, s.gsrc, s.nwords, s.bitpos);
                }
                my_tb = cd.start & ~(long long)(CO3_TILE - 1);
                my_lo = (int)(cd.start - my_tb);
                my_hi = my_lo + cd.len;
            }
            if (!all_mine && ttid < grp.count) {
                const Co3Chunk cd = chunk_of(grp.chunk0 + ttid);
                const long long tb = cd.start & ~(long long)(CO3_TILE - 1);
                tm.c_tb[gp][ttid] = tb;
                tm.c_lo[gp][ttid] = (int)(cd.start - tb);
                tm.c_hi[gp][ttid] = (int)(cd.start - tb) + cd.len;
            }
            // The bounds are read after the first quarter's barrier (and this set was last read two groups
            // ago); a warp stages and reads its own stream: no barrier is needed here.
#pragma unroll 1
            for (int q = 0; q < CO3_SUB / QB; ++q) {
                const int qoff = (q & 1) * accw;
                if (mine && s.active) {
                    const int a = max(s.i_lo, q * QB), b = min(s.i_hi, (q + 1) * QB);
                    if (b > a) {
                        const int row0 = qoff + ci * ACC_Q + (a - q * QB) * PADW + lane;
                        if (s.staged) decode_run<true>(r, lut_addr, acc_addr0 + 4u * (uint32_t)row0, b - a, tabs, bad);
                        else slow_run<true>(sr, tabs, s.gsrc, s.nwords, acc0 + row0, b - a, bad);
                    }
                }
                team_barrier(team);
                // read-out: warp w, round rr takes sub-chunk w + 8 rr, lane l its symbol q*QB + l; the
                // accumulator holds sum((K << 8) | length): the lengths of <= 8 users stay below 256
                const int e0 = warp * CO3_SUB + q * QB + lane;
                if (all_mine) {
                    read_out(acc0 + qoff + lane * PADW + warp, my_tb + e0, e0, my_lo, my_hi, scale, fu, inv_u, avg, weights, step);
                } else {
                    for (int cc = 0; cc < grp.count; ++cc)
                        read_out(acc0 + qoff + cc * ACC_Q + lane * PADW + warp, tm.c_tb[gp][cc] + e0, e0,
                                 tm.c_lo[gp][cc], tm.c_hi[gp][cc], scale, fu, inv_u, avg, weights, step);
                }
            }
            if (mine && s.active) {
                const uint32_t endpos = s.staged ? reader_pos(r, stage_addr) : sr.wp * 32u - (uint32_t)sr.nb;
                if (endpos - s.bitpos != s.sub_len_bits || endpos > s.nwords * 32u) bad = true;
            }
        }
        gi = ge;
    }
    if (bad) atomicOr(p.flags, CO3_FLAG_CORRUPT);
}

// ---- U = 1: nothing to add up, every warp on its own ------------------------------------------
// One user: a chunk is one stream, and the average is the stream's values themselves.  A block is 24
// independent warps that share the table; a warp stages its stream, decodes 32 symbols per lane at a
// time into a tile of its own (a plain store of the table entry: the cell is the lane's alone), and
// writes the tile out transposed, one 128-byte line of consecutive elements per store.  No barrier
// between warps except where the segment (the table) changes.  Lane s stores symbol i at word
// 33 i + s, the read-out lane i loads word 33 i + s of sub-chunk s: both free of bank conflicts.
constexpr int ONE_WARPS = 24, ONE_QB = 32, ONE_ROW = PADW, BITS_ONE = 12, ONE_DESC = 240;
struct SmemOne {
    TablesT<BITS_ONE> t;
    alignas(16) uint32_t stage[ONE_WARPS][STAGE_ROW];
    alignas(16) int32_t tile[ONE_WARPS][ONE_QB * ONE_ROW];
    Co3Chunk desc[ONE_DESC];                      // descriptors of the chunks of the current trip
};
static_assert(sizeof(SmemOne) + (4u << BITS_ONE) <= 227 * 1024, "one block per SM must fit its shared memory");

template <bool UPDATE>
__global__ void __launch_bounds__(ONE_WARPS * 32, 1)
decode_one_kernel(Co3Dev p, const uint32_t* __restrict__ bitstream, const uint16_t* __restrict__ sub_bits,
                  const uint32_t* __restrict__ chunk_off, const co3_seg_header* __restrict__ hdr,
                  float* __restrict__ avg, float* __restrict__ weights, float step) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    SmemOne& sm = *reinterpret_cast<SmemOne*>(s_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ __align__(16) uint32_t s_lut[1 << BITS_ONE];
    const unsigned char* lut_addr = reinterpret_cast<const unsigned char*>(s_lut);
    const uint32_t stage_addr = (uint32_t)__cvta_generic_to_shared(sm.stage[warp]);
    int32_t* tile = sm.tile[warp];
    const uint32_t tile_addr = (uint32_t)__cvta_generic_to_shared(tile);
    const int64_t c0 = p.dec_part[blockIdx.x], c1 = p.dec_part[blockIdx.x + 1];
    bool bad = false;
    for (int64_t i = tid; i < min(c1 - c0, (int64_t)ONE_DESC); i += ONE_WARPS * 32) sm.desc[i] = p.chunks[c0 + i];
    int64_t ci = c0;
    int loaded_seg = -1;
    while (ci < c1) {                              // one trip per run of at most ONE_DESC chunks of one segment
        const int seg = p.chunks[ci].seg;
        int64_t ce = ci + 1;
        while (ce < c1 && p.chunks[ce].seg == seg) ++ce;
        __syncthreads();                           // every warp is past its last look-up in the old tables and descriptors
        if (seg != loaded_seg) load_tables(sm.t, s_lut, p.cb, p.code_by_segment ? seg : co3_row_of(hdr[seg], &bad), tid, ONE_WARPS * 32);
        loaded_seg = seg;
        // The descriptors of the trip's chunks go to shared memory: the side information of a stream is
        // addressed through its descriptor, and with the descriptor in global memory every stream
        // waited for that load (110.6 -> 93.1 us on 2^26 elements).
        __syncthreads();
        const float scale = pow2_clamped((int)hdr[seg].bias + p.cF);
        // A warp's streams follow each other with their latencies taken apart: the side information of
        // the next stream (descriptor, offsets, its lane's sub-chunk length) is loaded while the current
        // one is decoded, and its payload copies are issued before the last read-out of the current one
        // (the stage is free once the last batch is decoded).
        struct Side { Co3Chunk cd; uint32_t w0, w1, sb; };
        auto fetch_side = [&](int64_t c) {
            Side x;
            x.cd = c - c0 < ONE_DESC ? sm.desc[c - c0] : p.chunks[c];
            const int lo = (int)(x.cd.start & (CO3_TILE - 1)), hi = lo + x.cd.len;
            const int sub_first = lo / CO3_SUB, sub_last = (hi - 1) / CO3_SUB;
            x.w0 = chunk_off[c];
            x.w1 = chunk_off[c + 1];
            x.sb = (lane >= sub_first && lane <= sub_last) ? sub_bits[x.cd.sub0 + (lane - sub_first)] : 0u;
            return x;
        };
        // offsets checked, payload copies issued (not waited for); returns the stream's word count
        auto issue_copies = [&](const Side& x, bool& staged, const uint32_t*& gsrc) {
            uint32_t nwords = 0;
            if ((x.w0 & 3u) || x.w1 < x.w0 || (int64_t)x.w1 > p.cap_words) bad = true;
            else nwords = x.w1 - x.w0;
            gsrc = bitstream + (nwords ? x.w0 : 0u);
            staged = nwords <= CO3_STAGE_WORDS;
            if (staged) {
                for (uint32_t i = lane; i < nwords / 4; i += 32)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(stage_addr + 16u * i), "l"(gsrc + 4u * i) : "memory");
                asm volatile("cp.async.commit_group;\n" ::: "memory");
            }
            return nwords;
        };
        int64_t c = ci + warp;
        Side cur;
        bool staged = true;
        const uint32_t* gsrc = bitstream;
        uint32_t nwords = 0;
        if (c < ce) {
            cur = fetch_side(c);
            nwords = issue_copies(cur, staged, gsrc);
        }
        while (c < ce) {
            const int64_t cn = c + ONE_WARPS;
            Side nxt = cur;
            if (cn < ce) nxt = fetch_side(cn);     // used only after this stream's last batch
            const Co3Chunk cd = cur.cd;
            const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
            const int lo = (int)(cd.start - tb), hi = lo + cd.len;
            Stream s;
            {
                const int sub_first = lo / CO3_SUB, sub_last = (hi - 1) / CO3_SUB;
                s.active = lane >= sub_first && lane <= sub_last;
                s.i_lo = max(lo - lane * CO3_SUB, 0);
                s.i_hi = min(hi - lane * CO3_SUB, CO3_SUB);
                s.nwords = nwords; s.staged = staged; s.gsrc = gsrc;
                uint32_t x = cur.sb;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
                    if (lane >= o) x += y;
                }
                s.bitpos = x - cur.sb;
                s.sub_len_bits = cur.sb;
                if (s.bitpos > nwords * 32u) { bad = true; s.bitpos = nwords * 32u; }
                asm volatile("cp.async.wait_group 0;\n" ::: "memory");
                __syncwarp();
            }
            Reader r;
            r.lo = 0; r.hi = 0; r.nb = 0; r.rp = stage_addr; r.nw = 0;
            SlowReader sr;
            sr.buf = 0; sr.nb = 0; sr.wp = 0;
            if (s.active) {
                if (s.staged) reader_init(r, stage_addr, s.bitpos);
                else slow_init(sr, s.gsrc, s.nwords, s.bitpos);
            }
            const bool whole = lo == 0 && hi == CO3_TILE;
            float* out = avg + tb + lane;           // element `lane` of the batch, sub-chunk 0
            float* wout = UPDATE ? weights + tb + lane : nullptr;
#pragma unroll 1
            for (int b = 0; b < CO3_SUB / ONE_QB; ++b) {
                if (s.active) {
                    const int a = max(s.i_lo, b * ONE_QB), z = min(s.i_hi, (b + 1) * ONE_QB);
                    if (z > a) {
                        const int cell = (a - b * ONE_QB) * ONE_ROW + lane;
                        if (s.staged) decode_run<true, TablesT<BITS_ONE>, true, ONE_ROW>(r, lut_addr, tile_addr + 4u * (uint32_t)cell, z - a, sm.t, bad);
                        else slow_run<true, TablesT<BITS_ONE>, true, ONE_ROW>(sr, sm.t, s.gsrc, s.nwords, tile + cell, z - a, bad);
                    }
                }
                __syncwarp();
                if (b == CO3_SUB / ONE_QB - 1) {   // the stream is decoded: check it, and let the next one's payload travel
                    if (s.active) {
                        const uint32_t endpos = s.staged ? reader_pos(r, stage_addr) : sr.wp * 32u - (uint32_t)sr.nb;
                        if (endpos - s.bitpos != s.sub_len_bits || endpos > s.nwords * 32u) bad = true;
                    }
                    if (cn < ce) nwords = issue_copies(nxt, staged, gsrc);
                }
                const int32_t* col = tile + lane * ONE_ROW;    // this lane's symbol of the batch, sub-chunk by sub-chunk
                if (whole) {
#pragma unroll 8
                    for (int sc = 0; sc < 32; ++sc) {
                        const float v = __fmul_rn((float)(col[sc] >> 8), scale);
                        out[sc * CO3_SUB] = v;
                        if (UPDATE) wout[sc * CO3_SUB] = __fadd_rn(wout[sc * CO3_SUB], __fmul_rn(step, v));
                    }
                } else {
                    for (int sc = 0; sc < 32; ++sc) {
                        const int e = sc * CO3_SUB + b * ONE_QB + lane;
                        if (e >= lo && e < hi) {
                            const float v = __fmul_rn((float)(col[sc] >> 8), scale);
                            out[sc * CO3_SUB] = v;
                            if (UPDATE) wout[sc * CO3_SUB] = __fadd_rn(wout[sc * CO3_SUB], __fmul_rn(step, v));
                        }
                    }
                }
                out += ONE_QB;
                if (UPDATE) wout += ONE_QB;
                __syncwarp();                      // the tile is written again by the next batch
            }
            cur = nxt;
            c = cn;
        }
        ci = ce;
    }
    if (bad) atomicOr(p.flags, CO3_FLAG_CORRUPT);
}

// ---- U > 8: whole-chunk accumulator, user groups of 8 --------------------------------------
// Teams as above (four, with a 12-bit table); a team decodes all users of one chunk into a
// whole-chunk accumulator, which the read-out leaves zeroed for the next chunk.
struct TeamB {
    alignas(16) int32_t acc[CO3_SUB * PADW];
    alignas(16) uint32_t stage[NW][STAGE_ROW];    // filled with 128-bit stores
};
constexpr int TEAMS_B = 4, BITS_B = 12;
struct SmemB {
    TablesT<BITS_B> t;
    TeamB team[TEAMS_B];
};
static_assert(sizeof(SmemB) + (4u << BITS_B) <= 227 * 1024, "one block per SM must fit its shared memory");

__global__ void __launch_bounds__(TEAMS_B * CO3_THREADS, 1)
decode_large_u_kernel(Co3Dev p, const uint32_t* __restrict__ bitstream,
                      const uint16_t* __restrict__ sub_bits, const uint32_t* __restrict__ chunk_off,
                      const co3_seg_header* __restrict__ hdr, float* __restrict__ avg,
                      float* __restrict__ weights, float step) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    SmemB& sm = *reinterpret_cast<SmemB*>(s_raw);
    const int tid = threadIdx.x, lane = tid & 31;
    const int team = tid / CO3_THREADS, ttid = tid - team * CO3_THREADS, warp = ttid >> 5;
    TeamB& tm = sm.team[team];
    __shared__ __align__(16) uint32_t s_lut[1 << BITS_B];
    const unsigned char* lut_addr = reinterpret_cast<const unsigned char*>(s_lut);
    const uint32_t acc_addr0 = (uint32_t)__cvta_generic_to_shared(tm.acc);
    const uint32_t stage_addr = (uint32_t)__cvta_generic_to_shared(tm.stage[warp]);
    const int64_t c0 = p.dec_part[blockIdx.x], c1 = p.dec_part[blockIdx.x + 1];
    const float fu = (float)p.U;
    const float inv_u = (p.U & (p.U - 1)) == 0 ? 1.0f / fu : 0.0f;
    bool bad = false;
    for (int i = ttid; i < CO3_SUB * PADW / 4; i += CO3_THREADS) reinterpret_cast<uint4*>(tm.acc)[i] = make_uint4(0, 0, 0, 0);
    int64_t ci = c0;
    while (ci < c1) {                              // one trip per run of chunks of one segment
        const int seg = p.chunks[ci].seg;
        int64_t ce = ci + 1;
        while (ce < c1 && p.chunks[ce].seg == seg) ++ce;
        __syncthreads();                           // every team is past its last look-up in the old tables
        load_tables(sm.t, s_lut, p.cb, p.code_by_segment ? seg : co3_row_of(hdr[seg], &bad), tid, TEAMS_B * CO3_THREADS);
        __syncthreads();                           // (and the first zeroing)
        const float scale = pow2_clamped((int)hdr[seg].bias + p.cF);
        for (int64_t c = ci + team; c < ce; c += TEAMS_B) {
            const Co3Chunk cd = p.chunks[c];
            for (int u = warp; u < p.U; u += NW) {
                Stream s;
                const uint32_t* co = chunk_off + (size_t)u * (p.n_chunks + 1) + c;
                open_stream(s, p, cd, c, u, bitstream, sub_bits, co[0], co[1], tm.stage[warp], lane, bad);
                if (s.active) {
                    const int row0 = s.i_lo * PADW + lane;
                    uint32_t endpos;
                    if (s.staged) {
                        Reader r;
                        reader_init(r, stage_addr, s.bitpos);
                        decode_run<false>(r, lut_addr, acc_addr0 + 4u * (uint32_t)row0, s.i_hi - s.i_lo, sm.t, bad);
                        endpos = reader_pos(r, stage_addr);
                    } else {
                        SlowReader sr;
                        slow_init(sr, s.gsrc, s.nwords, s.bitpos);
                        slow_run<false>(sr, sm.t, s.gsrc, s.nwords, tm.acc + row0, s.i_hi - s.i_lo, bad);
                        endpos = sr.wp * 32u - (uint32_t)sr.nb;
                    }
                    if (endpos - s.bitpos != s.sub_len_bits || endpos > s.nwords * 32u) bad = true;
                }
                __syncwarp();                      // the stage is reused by this warp's next user
            }
            team_barrier(team);
            const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
            const int lo = (int)(cd.start - tb), hi = lo + cd.len;
#pragma unroll 4
            for (int rr = 0; rr < CO3_TILE / CO3_THREADS; ++rr) {
                const int e = ttid + rr * CO3_THREADS;
                const int kk = e >> 7, il = e & (CO3_SUB - 1);
                const int32_t k = tm.acc[il * PADW + kk];
                tm.acc[il * PADW + kk] = 0;
                if (e >= lo && e < hi) put_out(avg, weights, step, tb + e, finish(k, scale, fu, inv_u));
            }
            team_barrier(team);
        }
        ci = ce;
    }
    if (bad) atomicOr(p.flags, CO3_FLAG_CORRUPT);
}

typedef void (*SmallKernel)(Co3Dev, const uint32_t*, const uint16_t*, const uint32_t*, const co3_seg_header*,
                            float*, float*, float);
struct SmallVariant {
    SmallKernel fn;
    int teams;
    size_t smem;                                  // dynamic shared memory
    size_t smem_static;                           // the primary table, the descriptors
};
// The widest table and the most teams that fit the shared memory of an SM (227 KB per block); user
// counts that do not divide 8 leave warps idle and keep the plain one-team blocks, four per SM.
SmallVariant small_variant(int U) {
    switch (U) {
        case 8: return {decode_small_u_kernel<4, 13, 8>, 4, smem_a_bytes<4, 13>(U), (4u << 13) + desc_bytes(8)};
        case 4: return {decode_small_u_kernel<4, 12, 4>, 4, smem_a_bytes<4, 12>(U), (4u << 12) + desc_bytes(4)};
        case 2: return {decode_small_u_kernel<3, 12, 2>, 3, smem_a_bytes<3, 12>(U), (4u << 12) + desc_bytes(2)};
        default: return {decode_small_u_kernel<1, CO3_LUT_SMALL_BITS, 0>, 1, smem_a_bytes<1, CO3_LUT_SMALL_BITS>(U), (4u << CO3_LUT_SMALL_BITS) + desc_bytes(0)};
    }
}

}  // namespace

cudaError_t co3_setup_decode_kernels(void) {
    for (int U = 1; U <= NW; ++U) {
        const SmallVariant v = small_variant(U);
        size_t need = v.smem;                      // the largest of the user counts that run this variant
        for (int U2 = 1; U2 <= NW; ++U2) {
            const SmallVariant v2 = small_variant(U2);
            if (v2.fn == v.fn && v2.smem > need) need = v2.smem;
        }
        if (need + v.smem_static > 227u * 1024u) return cudaErrorInvalidConfiguration;
        cudaError_t e = cudaFuncSetAttribute(v.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e1 = cudaFuncSetAttribute(decode_one_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SmemOne));
    if (e1 == cudaSuccess) e1 = cudaFuncSetAttribute(decode_one_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SmemOne));
    if (e1 != cudaSuccess) return e1;
    return cudaFuncSetAttribute(decode_large_u_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)sizeof(SmemB));
}

// Blocks the decoder of a plan with U users can keep resident: one block of several teams per SM, or
// (user counts that do not divide 8) as many one-team blocks as fit.
int co3_decode_max_blocks(int U, int num_sms) {
    if (U > NW || U == 1) return num_sms;
    const SmallVariant v = small_variant(U);
    int bpsm = 1;
    if (v.teams == 1) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bpsm, v.fn, CO3_THREADS, v.smem) != cudaSuccess) (void)cudaGetLastError();
        if (bpsm < 1) bpsm = 1;
    }
    return num_sms * bpsm;
}

// The decoder's work items (groups of chunks for U <= 8, chunks above) with their segment and a cost
// in team-rounds (1 = a chunk whose longest sub-chunk is full), split over the blocks by
// co3_host_balanced_split.
int co3_decode_partition(const Co3Chunk* chunks, int64_t n_chunks, const Co3Group* groups, int64_t n_groups, int U,
                         int max_blocks, int32_t* part) {
    const bool by_group = U <= NW && U > 1;        // one user: chunks, taken by 32 independent warps
    const int teams = U == 1 ? ONE_WARPS : (by_group ? small_variant(U).teams : TEAMS_B);
    const int64_t n = by_group ? n_groups : n_chunks;
    double* w = (double*)malloc(sizeof(double) * (size_t)n);
    int32_t* seg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    int blocks = -1;
    if (w && seg) {
        for (int64_t i = 0; i < n; ++i) {
            int longest = 0;
            if (by_group) {
                seg[i] = groups[i].seg;
                for (int k = 0; k < groups[i].count; ++k) {
                    const int len = chunks[groups[i].chunk0 + k].len;
                    longest = longest > len ? longest : len;
                }
            } else {
                seg[i] = chunks[i].seg;
                longest = chunks[i].len;
            }
            w[i] = 0.04 + (longest >= CO3_SUB ? 1.0 : (double)longest / CO3_SUB);
        }
        blocks = co3_host_balanced_split(w, seg, n, teams, max_blocks, 0.08, part);
    }
    free(w); free(seg);
    return blocks;
}

cudaError_t co3_launch_decode(co3_plan* pl, const uint32_t* bitstream, const uint16_t* sub_bits,
                              const uint32_t* chunk_off, const co3_seg_header* hdr, float* avg,
                              float* weights, float step, cudaStream_t st) {
    Co3Dev p = pl->dev;
    if (pl->cfg.bias_mode == CO3_CODE_EMPIRICAL) { p.cb = pl->cb_emp; p.code_by_segment = 1; }
    co3_prof_begin(pl, CO3_K_DECODE, st);
    if (p.U == 1) {
        if (weights) decode_one_kernel<true><<<p.dec_blocks, ONE_WARPS * 32, sizeof(SmemOne), st>>>(p, bitstream, sub_bits, chunk_off, hdr, avg, weights, step);
        else decode_one_kernel<false><<<p.dec_blocks, ONE_WARPS * 32, sizeof(SmemOne), st>>>(p, bitstream, sub_bits, chunk_off, hdr, avg, weights, step);
    } else if (p.U <= NW) {
        const SmallVariant v = small_variant(p.U);
        v.fn<<<p.dec_blocks, v.teams * CO3_THREADS, v.smem, st>>>(p, bitstream, sub_bits, chunk_off, hdr, avg, weights, step);
    } else {
        decode_large_u_kernel<<<p.dec_blocks, TEAMS_B * CO3_THREADS, sizeof(SmemB), st>>>(
            p, bitstream, sub_bits, chunk_off, hdr, avg, weights, step);
    }
    co3_prof_end(pl, CO3_K_DECODE, st, 1);
    return cudaGetLastError();
}
