// h_Hf on the device (Algorithm 1 line 9): Huffman-code the converted symbols of every user
// into the chunked container.  Three launches, no device-side waiting:
//   1. enc_len_kernel  -- code length of every symbol -> bits per sub-chunk and words per chunk
//   2. enc_scan_kernel -- exclusive scan of the chunk word counts per user -> chunk offsets,
//                         capacity check before anything is written
//   3. enc_pack_kernel -- per chunk: per-thread bit offsets by a block scan, codewords merged
//                         into a shared-memory image of the chunk, 128-bit coalesced stores
// Work item = (user, chunk); a thread owns 16 consecutive symbols (one 128-bit load), 8 threads
// own a sub-chunk, a block owns a chunk.  Blocks are persistent over contiguous item ranges, keep
// the segment's table in shared memory (replicated once per lane, so the look-ups are free of
// bank conflicts) and always have the next item's symbols in flight.  In the pack kernel a thread
// first merges its 16 codewords pairwise in registers (16 -> 8 -> 4 pieces of at most 64 bits),
// then ORs the four pieces into the chunk image at its scanned bit offset.
// Bound: HBM for the symbol reads (1 B/element, twice) and payload writes (~0.85 B/element), with
// integer issue slots and shared-memory look-ups (one per symbol per pass) close behind.
#include "co3_internal.h"

namespace {

constexpr int BUF_WORDS = CO3_TILE * CO3_MAXLEN / 32;   // 2048: a chunk at 16 bits per symbol

struct Item {                    // one (user, chunk) work item as a thread sees it
    uint32_t u, c;
    uint32_t w[4];               // this thread's 16 symbols
    uint32_t mask;               // which of them belong to the chunk
    uint32_t dst_word, skip;     // pack pass: the chunk's word offset; user's payload does not fit
};

// Cursor over a block's contiguous item range in (user, chunk) order.  (Contiguous, not
// interleaved across blocks: a block then changes segment -- and reloads its replicated table --
// only a few times.)
struct Cursor {
    uint32_t next, end, u, c, n_chunks;
    __device__ __forceinline__ bool more() const { return next < end; }
    __device__ __forceinline__ void advance() {
        ++next;
        if (++c == n_chunks) { c = 0; ++u; }
    }
};

__device__ __forceinline__ void fetch_item(Item& it, const Co3Dev& p, uint32_t u, uint32_t c, int tid) {
    it.u = u;
    it.c = c;
    const Co3Chunk cd = p.chunks[c];
    const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
    const int lo = (int)(cd.start - tb), hi = lo + cd.len;
    const int e0 = 16 * tid;
    it.mask = 0;
    it.w[0] = it.w[1] = it.w[2] = it.w[3] = 0;
    if (e0 < hi && e0 + 16 > lo) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p.sym + (size_t)u * p.sld + tb + e0));
        it.w[0] = v.x; it.w[1] = v.y; it.w[2] = v.z; it.w[3] = v.w;
        const int a = max(lo - e0, 0), b = min(hi - e0, 16);     // valid bytes [a, b)
        it.mask = (b >= 16 ? 0xFFFFu : ((1u << b) - 1u)) & ~((1u << a) - 1u);
    }
}

// Look up the 16 table entries of a thread's symbols; entries of masked-out symbols are 0.
__device__ __forceinline__ void lookup16(const uint32_t* s_tab, int lane, const uint32_t w[4],
                                         uint32_t mask, uint32_t ent[16]) {
    if (mask == 0xFFFFu) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t s = __byte_perm(w[i >> 2], 0, 0x4440 + (i & 3));
            ent[i] = s_tab[s * 32 + lane];
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t s = __byte_perm(w[i >> 2], 0, 0x4440 + (i & 3));
            ent[i] = ((mask >> i) & 1u) ? s_tab[s * 32 + lane] : 0u;
        }
    }
}

__device__ __forceinline__ void cursor_init(Cursor& cu, const Co3Dev& p) {
    cu.n_chunks = (uint32_t)p.n_chunks;
    const uint32_t n_items = cu.n_chunks * (uint32_t)p.U;
    const uint32_t per = (n_items + gridDim.x - 1) / gridDim.x;
    cu.next = blockIdx.x * per;
    cu.end = min(n_items, cu.next + per);
    cu.u = cu.next / cu.n_chunks;
    cu.c = cu.next - cu.u * cu.n_chunks;
}

__global__ void __launch_bounds__(CO3_THREADS)
enc_len_kernel(Co3Dev p, const co3_seg_header* __restrict__ hdr, uint16_t* __restrict__ sub_bits) {
    extern __shared__ __align__(16) uint32_t s_dyn[];
    uint32_t* s_len = s_dyn;                          // [nsym][32 lanes] code lengths
    __shared__ uint32_t s_warp[2][CO3_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    Cursor cu;
    cursor_init(cu, p);
    if (!cu.more()) return;
    int cur_seg = -1, par = 0;
    bool bad = false;

    auto process = [&](const Item& cur, uint32_t item) {
        const Co3Chunk cd = p.chunks[cur.c];
        if (cd.seg != cur_seg) {
            __syncthreads();
            const uint8_t* src = p.cb.len8 + (size_t)co3_row_of(hdr[cd.seg], &bad) * CO3_MAXSYM;
            for (int i = tid; i < p.nsym * 32; i += CO3_THREADS) s_len[i] = src[i >> 5];
            cur_seg = cd.seg;
            __syncthreads();
        }
        uint32_t ent[16];
        lookup16(s_len, lane, cur.w, cur.mask, ent);
        uint32_t bits = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) bits += ent[i];
        // 8 threads = one sub-chunk
        uint32_t sb = bits;
        sb += __shfl_xor_sync(0xffffffffu, sb, 1);
        sb += __shfl_xor_sync(0xffffffffu, sb, 2);
        sb += __shfl_xor_sync(0xffffffffu, sb, 4);
        const int tlo = (int)(cd.start & (CO3_TILE - 1));
        const int sub_first = tlo / CO3_SUB, sub_last = (tlo + cd.len - 1) / CO3_SUB;
        const int kk = tid >> 3;
        if ((tid & 7) == 0 && kk >= sub_first && kk <= sub_last)
            sub_bits[(size_t)cur.u * p.n_sub + cd.sub0 + (kk - sub_first)] = (uint16_t)sb;
        uint32_t wb = ((lane & 7) == 0) ? sb : 0u;     // every lane of a sub-chunk holds sb: count it once
        wb += __shfl_xor_sync(0xffffffffu, wb, 8);
        wb += __shfl_xor_sync(0xffffffffu, wb, 16);
        par ^= 1;
        if (lane == 0) s_warp[par][warp] = wb;
        __syncthreads();
        if (tid == 0) {
            uint32_t tot = 0;
#pragma unroll
            for (int k = 0; k < CO3_THREADS / 32; ++k) tot += s_warp[par][k];
            p.chunk_words[item] = 4u * ((tot + 127u) / 128u);
            p.chunk_bits[item] = tot;
        }
    };

    // two item buffers used alternately, so that the next item's loads stay in flight while the
    // current one is processed (no register copies that would wait for them)
    Item a, b;
    fetch_item(a, p, cu.u, cu.c, tid);
    while (true) {
        const uint32_t ia = cu.next;
        cu.advance();
        if (cu.more()) fetch_item(b, p, cu.u, cu.c, tid);
        process(a, ia);
        if (!cu.more()) break;
        const uint32_t ib = cu.next;
        cu.advance();
        if (cu.more()) fetch_item(a, p, cu.u, cu.c, tid);
        process(b, ib);
        if (!cu.more()) break;
    }
    if (bad && tid == 0) atomicOr(p.flags, CO3_FLAG_CORRUPT);
}

// chunk_off[u][c] = exclusive prefix of the chunk word counts of user u; one block per user.
__global__ void __launch_bounds__(1024)
enc_scan_kernel(Co3Dev p, uint32_t* __restrict__ chunk_off, unsigned long long* __restrict__ user_bits) {
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_carry;
    __shared__ unsigned long long s_bits[32];
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t* in = p.chunk_words + (size_t)u * p.n_chunks;
    const uint32_t* inb = p.chunk_bits + (size_t)u * p.n_chunks;
    uint32_t* out = chunk_off + (size_t)u * (p.n_chunks + 1);
    unsigned long long my_bits = 0;                   // r_t^(u): code bits of this user
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < p.n_chunks; base += 1024) {
        const int64_t i = base + tid;
        const uint32_t v = (i < p.n_chunks) ? in[i] : 0u;
        my_bits += (i < p.n_chunks) ? inb[i] : 0u;
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

__global__ void __launch_bounds__(CO3_THREADS)
enc_pack_kernel(Co3Dev p, const co3_seg_header* __restrict__ hdr, const uint32_t* __restrict__ chunk_off,
                uint32_t* __restrict__ bitstream) {
    extern __shared__ __align__(16) uint32_t s_dyn[];
    uint32_t* s_enc = s_dyn;                          // [nsym][32 lanes] codeword | length << 16
    uint32_t* s_buf = s_dyn + p.nsym * 32;            // BUF_WORDS + 4
    __shared__ uint32_t s_warp[2][CO3_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    Cursor cu;
    cursor_init(cu, p);
    if (!cu.more()) return;
    int cur_seg = -1, par = 0;
    bool bad = false;
    uint32_t prev_words = BUF_WORDS + 4;              // words of the image that may be non-zero

    auto fetch = [&](Item& it) {
        fetch_item(it, p, cu.u, cu.c, tid);
        it.skip = p.user_ovf[cu.u];
        it.dst_word = chunk_off[(size_t)cu.u * (cu.n_chunks + 1) + cu.c];
    };
    auto process = [&](const Item& cur, uint32_t item) {
        if (cur.skip) return;                         // block-uniform: this user's payload does not fit
        const int seg = p.chunks[cur.c].seg;
        if (seg != cur_seg) {
            const uint32_t* src = p.cb.enc + (size_t)co3_row_of(hdr[seg], &bad) * CO3_MAXSYM;
            for (int i = tid; i < p.nsym * 32; i += CO3_THREADS) s_enc[i] = src[i >> 5];
            cur_seg = seg;
        }
        {   // clear what the previous chunk left in the image (all of it the first time)
            uint4* z = reinterpret_cast<uint4*>(s_buf);
            for (uint32_t i = tid; i < (prev_words + 3) / 4; i += CO3_THREADS) z[i] = make_uint4(0, 0, 0, 0);
        }
        __syncthreads();                              // table and cleared image visible
        uint32_t ent[16];
        lookup16(s_enc, lane, cur.w, cur.mask, ent);
        // merge 16 codewords -> 8 pieces (<= 32 bits) -> 4 pieces (<= 64 bits)
        uint32_t c1[8], l1[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t x0 = ent[2 * k], x1 = ent[2 * k + 1];
            c1[k] = (x0 & 0xFFFFu) | ((x1 & 0xFFFFu) << (x0 >> 16));
            l1[k] = (x0 >> 16) + (x1 >> 16);
        }
        unsigned long long c2[4];
        uint32_t l2[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            c2[k] = (unsigned long long)c1[2 * k] | ((unsigned long long)c1[2 * k + 1] << l1[2 * k]);
            l2[k] = l1[2 * k] + l1[2 * k + 1];
        }
        const uint32_t bits = l2[0] + l2[1] + l2[2] + l2[3];
        // exclusive scan of the per-thread bit counts over the block
        uint32_t x = bits;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        par ^= 1;
        if (lane == 31) s_warp[par][warp] = x;
        __syncthreads();
        uint32_t pre = 0, total = 0;
#pragma unroll
        for (int k = 0; k < CO3_THREADS / 32; ++k) {
            const uint32_t t = s_warp[par][k];
            pre += (k < warp) ? t : 0u;
            total += t;
        }
        const uint32_t nwords = 4u * ((total + 127u) / 128u);
        uint32_t pos = pre + x - bits;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            put_piece(s_buf, pos, c2[k]);
            pos += l2[k];
        }
        __syncthreads();
        uint4* dst = reinterpret_cast<uint4*>(bitstream + (size_t)cur.u * p.cap_words + cur.dst_word);
        const uint4* srcv = reinterpret_cast<const uint4*>(s_buf);
        for (uint32_t i = tid; i < nwords / 4; i += CO3_THREADS) dst[i] = srcv[i];
        prev_words = nwords;
        __syncthreads();
    };

    Item a, b;
    fetch(a);
    while (true) {
        const uint32_t ia = cu.next;
        cu.advance();
        if (cu.more()) fetch(b);
        process(a, ia);
        if (!cu.more()) break;
        const uint32_t ib = cu.next;
        cu.advance();
        if (cu.more()) fetch(a);
        process(b, ib);
        if (!cu.more()) break;
    }
    if (bad && tid == 0) atomicOr(p.flags, CO3_FLAG_CORRUPT);
}

int g_len_bpsm[4] = {0, 0, 0, 0}, g_pack_bpsm[4] = {0, 0, 0, 0};

}  // namespace

cudaError_t co3_setup_kernels(void) {
    cudaError_t e = cudaFuncSetAttribute(enc_pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (CO3_MAXSYM * 32 + BUF_WORDS + 4) * (int)sizeof(uint32_t));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(enc_len_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                CO3_MAXSYM * 32 * (int)sizeof(uint32_t));
}

cudaError_t co3_launch_encode(co3_plan* pl, const co3_seg_header* hdr, uint32_t* bitstream,
                              uint16_t* sub_bits, uint32_t* chunk_off, unsigned long long* user_bits,
                              cudaStream_t st) {
    const Co3Dev& p = pl->dev;
    const int64_t items = p.n_chunks * (int64_t)p.U;
    cudaError_t e = cudaSuccess;
    const int fi = p.nsym == 256 ? 0 : (p.nsym == 128 ? 1 : (p.nsym == 64 ? 2 : 3));
    const size_t smem_len = (size_t)p.nsym * 32 * sizeof(uint32_t);
    if (!g_len_bpsm[fi]) {
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_len_bpsm[fi], enc_len_kernel, CO3_THREADS, smem_len);
        if (g_len_bpsm[fi] < 1) g_len_bpsm[fi] = 1;
    }
    int64_t grid = (int64_t)pl->num_sms * g_len_bpsm[fi];
    co3_prof_begin(pl, CO3_K_ENC_LEN, st);
    enc_len_kernel<<<(int)(items < grid ? items : grid), CO3_THREADS, smem_len, st>>>(p, hdr, sub_bits);
    co3_prof_end(pl, CO3_K_ENC_LEN, st, 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    co3_prof_begin(pl, CO3_K_ENC_SCAN, st);
    enc_scan_kernel<<<p.U, 1024, 0, st>>>(p, chunk_off, user_bits);
    co3_prof_end(pl, CO3_K_ENC_SCAN, st, 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const size_t smem = ((size_t)p.nsym * 32 + BUF_WORDS + 4) * sizeof(uint32_t);
    if (!g_pack_bpsm[fi]) {
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_pack_bpsm[fi], enc_pack_kernel, CO3_THREADS, smem);
        if (g_pack_bpsm[fi] < 1) g_pack_bpsm[fi] = 1;
    }
    grid = (int64_t)pl->num_sms * g_pack_bpsm[fi];
    co3_prof_begin(pl, CO3_K_ENC_PACK, st);
    enc_pack_kernel<<<(int)(items < grid ? items : grid), CO3_THREADS, smem, st>>>(p, hdr, chunk_off, bitstream);
    co3_prof_end(pl, CO3_K_ENC_PACK, st, 1);
    return cudaGetLastError();
}
