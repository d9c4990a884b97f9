// h_Hf on the device (Algorithm 1 line 9): Huffman-code the converted symbols of every user
// into the chunked container.  Three launches, no device-side waiting:
//   1. enc_len_kernel  -- code length of every symbol -> bits per sub-chunk and words per chunk
//   2. enc_scan_kernel -- exclusive scan of the chunk word counts per user -> chunk offsets,
//                         capacity check before anything is written
//   3. enc_pack_kernel -- per chunk: per-thread bit offsets by a block scan, codewords merged
//                         into a shared-memory image of the chunk, 128-bit coalesced stores
// Work item = (user, chunk); a thread owns 16 consecutive symbols (one 128-bit load), 8 threads
// own a sub-chunk, a block owns a chunk.  Blocks are persistent over contiguous item ranges and
// keep the segment's code table in shared memory, replicated once per lane so that the table
// look-ups are free of bank conflicts.  Bound: HBM for the symbol reads (1 B/element, twice) and
// payload writes (~0.85 B/element), with integer issue slots close behind.
#include "co3_internal.h"

namespace {

constexpr int BUF_WORDS = CO3_TILE * CO3_MAXLEN / 32;   // 2048: a chunk at 16 bits per symbol

__device__ __forceinline__ void load_symbols(const Co3Dev& p, int u, const Co3Chunk& cd, int tid,
                                             uint32_t w[4], uint32_t& mask) {
    const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
    const int lo = (int)(cd.start - tb), hi = lo + cd.len;
    const int e0 = 16 * tid;
    mask = 0;
    w[0] = w[1] = w[2] = w[3] = 0;
    if (e0 < hi && e0 + 16 > lo) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p.sym + (size_t)u * p.sld + tb + e0));
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
        const int a = max(lo - e0, 0), b = min(hi - e0, 16);     // valid bytes [a, b)
        mask = (b >= 16 ? 0xFFFFu : ((1u << b) - 1u)) & ~((1u << a) - 1u);
    }
}

__global__ void __launch_bounds__(CO3_THREADS)
enc_len_kernel(Co3Dev p, Co3CodeBook cb, uint16_t* __restrict__ sub_bits, unsigned long long* user_bits) {
    __shared__ uint32_t s_len[(CO3_MAXSYM / 4) * 32];   // [word of 4 lengths][lane]
    __shared__ uint32_t s_warp[CO3_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t n_items = p.n_chunks * (int64_t)p.U;
    const int64_t per = (n_items + gridDim.x - 1) / gridDim.x;
    const int64_t it0 = (int64_t)blockIdx.x * per, it1 = min(n_items, it0 + per);
    int cur_seg = -1;
    for (int64_t item = it0; item < it1; ++item) {
        const int u = (int)(item / p.n_chunks);
        const int64_t c = item - (int64_t)u * p.n_chunks;
        const Co3Chunk cd = p.chunks[c];
        if (cd.seg != cur_seg) {
            __syncthreads();
            const uint32_t* src = reinterpret_cast<const uint32_t*>(cb.len8 + (size_t)cd.seg * CO3_MAXSYM);
            for (int i = tid; i < (p.nsym / 4) * 32; i += CO3_THREADS) s_len[i] = src[i >> 5];
            cur_seg = cd.seg;
            __syncthreads();
        }
        uint32_t w[4], mask;
        load_symbols(p, u, cd, tid, w, mask);
        uint32_t bits = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t s = (w[i >> 2] >> (8 * (i & 3))) & 0xFFu;
            const uint32_t l4 = s_len[(s >> 2) * 32 + lane];
            const uint32_t l = (l4 >> (8 * (s & 3))) & 0xFFu;
            bits += ((mask >> i) & 1u) ? l : 0u;
        }
        // 8 threads = one sub-chunk
        uint32_t sb = bits;
        sb += __shfl_xor_sync(0xffffffffu, sb, 1);
        sb += __shfl_xor_sync(0xffffffffu, sb, 2);
        sb += __shfl_xor_sync(0xffffffffu, sb, 4);
        const int64_t tb = cd.start & ~(int64_t)(CO3_TILE - 1);
        const int sub_first = (int)((cd.start - tb) / CO3_SUB);
        const int sub_last = (int)((cd.start - tb + cd.len - 1) / CO3_SUB);
        const int kk = tid >> 3;
        if ((tid & 7) == 0 && kk >= sub_first && kk <= sub_last)
            sub_bits[(size_t)u * p.n_sub + cd.sub0 + (kk - sub_first)] = (uint16_t)sb;
        uint32_t wb = sb;                       // every lane of a sub-chunk holds sb: count it once
        wb = ((lane & 7) == 0) ? wb : 0u;
        wb += __shfl_xor_sync(0xffffffffu, wb, 8);
        wb += __shfl_xor_sync(0xffffffffu, wb, 16);
        if (lane == 0) s_warp[warp] = wb;
        __syncthreads();
        if (tid == 0) {
            uint32_t tot = 0;
#pragma unroll
            for (int k = 0; k < CO3_THREADS / 32; ++k) tot += s_warp[k];
            p.chunk_words[item] = 4u * ((tot + 127u) / 128u);
            atomicAdd(&user_bits[u], (unsigned long long)tot);
        }
        __syncthreads();
    }
}

// chunk_off[u][c] = exclusive prefix of the chunk word counts of user u; one block per user.
__global__ void __launch_bounds__(1024) enc_scan_kernel(Co3Dev p, uint32_t* __restrict__ chunk_off) {
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_carry;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t* in = p.chunk_words + (size_t)u * p.n_chunks;
    uint32_t* out = chunk_off + (size_t)u * (p.n_chunks + 1);
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < p.n_chunks; base += 1024) {
        const int64_t i = base + tid;
        const uint32_t v = (i < p.n_chunks) ? in[i] : 0u;
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
    if (tid == 0) {
        const uint32_t total = s_carry;
        out[p.n_chunks] = total;
        const uint32_t ovf = (int64_t)total > p.cap_words;
        p.user_ovf[u] = ovf;
        if (ovf) atomicOr(p.flags, CO3_FLAG_CAPACITY);
    }
}

__global__ void __launch_bounds__(CO3_THREADS)
enc_pack_kernel(Co3Dev p, Co3CodeBook cb, const uint32_t* __restrict__ chunk_off, uint32_t* __restrict__ bitstream) {
    extern __shared__ __align__(16) uint32_t s_dyn[];
    uint32_t* s_enc = s_dyn;                          // [nsym][32 lanes]
    uint32_t* s_buf = s_dyn + p.nsym * 32;            // BUF_WORDS + 4
    __shared__ uint32_t s_warp[CO3_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t n_items = p.n_chunks * (int64_t)p.U;
    const int64_t per = (n_items + gridDim.x - 1) / gridDim.x;
    const int64_t it0 = (int64_t)blockIdx.x * per, it1 = min(n_items, it0 + per);
    int cur_seg = -1;
    for (int64_t item = it0; item < it1; ++item) {
        const int u = (int)(item / p.n_chunks);
        const int64_t c = item - (int64_t)u * p.n_chunks;
        if (p.user_ovf[u]) continue;                  // block-uniform
        const Co3Chunk cd = p.chunks[c];
        if (cd.seg != cur_seg) {
            __syncthreads();
            const uint32_t* src = cb.enc + (size_t)cd.seg * CO3_MAXSYM;
            for (int i = tid; i < p.nsym * 32; i += CO3_THREADS) s_enc[i] = src[i >> 5];
            cur_seg = cd.seg;
            __syncthreads();
        }
        uint32_t w[4], mask;
        load_symbols(p, u, cd, tid, w, mask);
        uint32_t ent[16];
        uint32_t bits = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t s = (w[i >> 2] >> (8 * (i & 3))) & 0xFFu;
            const uint32_t e = s_enc[s * 32 + lane];
            ent[i] = ((mask >> i) & 1u) ? e : 0u;
            bits += ent[i] >> 16;
        }
        // exclusive scan of the per-thread bit counts over the block
        uint32_t x = bits;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) s_warp[warp] = x;
        __syncthreads();
        uint32_t pre = 0, total = 0;
#pragma unroll
        for (int k = 0; k < CO3_THREADS / 32; ++k) {
            const uint32_t t = s_warp[k];
            pre += (k < warp) ? t : 0u;
            total += t;
        }
        const uint32_t nwords = 4u * ((total + 127u) / 128u);
        for (uint32_t i = tid; i < nwords; i += CO3_THREADS) s_buf[i] = 0;
        __syncthreads();
        uint32_t pos = pre + x - bits;
        uint32_t wi = pos >> 5, nb = pos & 31u;
        unsigned long long acc = 0;
        bool first = true;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            acc |= (unsigned long long)(ent[i] & 0xFFFFu) << nb;
            nb += ent[i] >> 16;
            if (nb >= 32u) {
                if (first) { atomicOr(&s_buf[wi], (uint32_t)acc); first = false; }
                else s_buf[wi] = (uint32_t)acc;        // a word wholly inside this thread's span
                acc >>= 32; nb -= 32u; ++wi;
            }
        }
        if (acc) atomicOr(&s_buf[wi], (uint32_t)acc);
        __syncthreads();
        uint4* dst = reinterpret_cast<uint4*>(bitstream + (size_t)u * p.cap_words +
                                              chunk_off[(size_t)u * (p.n_chunks + 1) + c]);
        const uint4* srcv = reinterpret_cast<const uint4*>(s_buf);
        for (uint32_t i = tid; i < nwords / 4; i += CO3_THREADS) dst[i] = srcv[i];
        __syncthreads();
    }
}

int g_len_bpsm = 0, g_pack_bpsm[4] = {0, 0, 0, 0};

}  // namespace

cudaError_t co3_setup_kernels(void) {
    return cudaFuncSetAttribute(enc_pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (CO3_MAXSYM * 32 + BUF_WORDS + 4) * (int)sizeof(uint32_t));
}

cudaError_t co3_launch_encode(co3_plan* pl, uint32_t* bitstream, uint16_t* sub_bits,
                              uint32_t* chunk_off, unsigned long long* user_bits, cudaStream_t st) {
    const Co3Dev& p = pl->dev;
    const int64_t items = p.n_chunks * (int64_t)p.U;
    cudaError_t e = cudaMemsetAsync(user_bits, 0, sizeof(unsigned long long) * (size_t)p.U, st);
    if (e != cudaSuccess) return e;
    if (!g_len_bpsm) {
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_len_bpsm, enc_len_kernel, CO3_THREADS, 0);
        if (g_len_bpsm < 1) g_len_bpsm = 1;
    }
    int64_t grid = (int64_t)pl->num_sms * g_len_bpsm;
    co3_prof_begin(pl, CO3_K_ENC_LEN, st);
    enc_len_kernel<<<(int)(items < grid ? items : grid), CO3_THREADS, 0, st>>>(p, pl->cb_enc, sub_bits, user_bits);
    co3_prof_end(pl, CO3_K_ENC_LEN, st, 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    co3_prof_begin(pl, CO3_K_ENC_SCAN, st);
    enc_scan_kernel<<<p.U, 1024, 0, st>>>(p, chunk_off);
    co3_prof_end(pl, CO3_K_ENC_SCAN, st, 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const size_t smem = ((size_t)p.nsym * 32 + BUF_WORDS + 4) * sizeof(uint32_t);
    const int fi = p.nsym == 256 ? 0 : (p.nsym == 128 ? 1 : (p.nsym == 64 ? 2 : 3));
    if (!g_pack_bpsm[fi]) {
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_pack_bpsm[fi], enc_pack_kernel, CO3_THREADS, smem);
        if (g_pack_bpsm[fi] < 1) g_pack_bpsm[fi] = 1;
    }
    grid = (int64_t)pl->num_sms * g_pack_bpsm[fi];
    co3_prof_begin(pl, CO3_K_ENC_PACK, st);
    enc_pack_kernel<<<(int)(items < grid ? items : grid), CO3_THREADS, smem, st>>>(p, pl->cb_enc, chunk_off, bitstream);
    co3_prof_end(pl, CO3_K_ENC_PACK, st, 1);
    return cudaGetLastError();
}
