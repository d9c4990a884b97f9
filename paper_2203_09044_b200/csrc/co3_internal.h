// Internal declarations of the CO3 CUDA library (sm_100a).  Not part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "co3.h"

constexpr int CO3_TILE = 4096;      // chunk grid (elements)
constexpr int CO3_SUB = 128;        // sub-chunk grid (elements)
constexpr int CO3_MAXLEN = 16;      // longest codeword
constexpr int CO3_LUT_BITS = 13;    // index width of the stored primary decode tables
constexpr int CO3_LUT_SIZE = 1 << CO3_LUT_BITS;
constexpr int CO3_LUT_SMALL_BITS = 11;  // a decoder short of shared memory keeps the first 2^11 entries
                                        // (minus those of longer codewords: the table is indexed LSB-first)
constexpr int CO3_LONG_FROM = CO3_LUT_SMALL_BITS + 1;   // shortest codeword the second table holds
constexpr int CO3_NCAND = 10;       // model codes: weight floors 2^0 .. 2^9 tried in parallel (weights sum to ~2^20: 2^9 always passes)
constexpr int CO3_NCAND_HIST = 32;  // codes from counts (total below 2^31): floors 2^0 .. 2^31 (2^31 makes all weights equal)
constexpr int CO3_NIBETA = 23;      // ibeta in [-14, 8]
constexpr int CO3_NIR = 128;        // ir in [-96, 31]
constexpr int CO3_IBETA_MIN = -14, CO3_IBETA_MAX = 8, CO3_IR_MIN = -96, CO3_IR_MAX = 31;
constexpr int CO3_NROWS = CO3_NIBETA * CO3_NIR;   // model rows (codes) per format
constexpr int CO3_FIT_GRID = 8192;  // log R(beta) is tabulated at FIT_GRID + 1 points, uniform in log2 beta
constexpr int CO3_MAXSYM = 256;     // alphabet rows are padded to 256 entries
constexpr int CO3_STAGE_WORDS = 1024;  // shared-memory staging per (chunk, user) stream in decode
constexpr int CO3_THREADS = 256;
constexpr int CO3_SUB_WORDS = CO3_SUB * CO3_MAXLEN / 32;     // payload words of a sub-chunk at 16 bits per symbol (64)
constexpr int CO3_SLOT_WORDS = CO3_TILE * CO3_MAXLEN / 32;   // ... of a chunk (2048)

// One chunk of the static partition: elements [start, start+len) of every user's row, all in
// segment `seg`, inside one 4096-aligned tile.  sub0 = index of its first sub-chunk.
struct Co3Chunk {
    int64_t start;
    int32_t len;
    int32_t seg;
    int32_t sub0;
    int32_t pad_;
};

// A group of consecutive chunks of one segment decoded together by one block (U <= 8).
struct Co3Group {
    int32_t chunk0;
    int32_t count;
    int32_t seg;
    int32_t pad_;
};

// Code tables for every model row r = (ibeta - IBETA_MIN) * NIR + (ir - IR_MIN).  The Huffman
// code of a segment is a pure function of the format and of the two header indices, so all
// CO3_NROWS codes are built on the device once, when the plan is created; an iteration only
// selects rows.  Rows are CO3_MAXSYM / CO3_LUT_SIZE wide.
// entries of lut_long that the decoder keeps in shared memory
constexpr int CO3_LONG_CACHE = 512;

struct Co3CodeBook {
    int ncand;           //                 weight-floor candidates of this book (NCAND or NCAND_HIST)
    uint8_t* cand_len;   // [R][ncand][256] code lengths per weight-floor candidate (build scratch)
    int32_t* cand_max;   // [R][ncand]      longest codeword per candidate (build scratch)
    uint8_t* len8;       // [R][256]        chosen lengths, by internal symbol
    uint8_t* len_pub;    // [R][256]        the same by public symbol (inspection only)
    uint32_t* enc;       // [R][256]        bit-reversed codeword | length << 16, by internal symbol
    uint32_t* code_msb;  // [R][256]        canonical codeword, root bit most significant, by public symbol
    uint32_t* lut;       // [R][8192]       (signed magnitude << 8) | length, 0 = longer than 13 bits
    uint32_t* lut_long;  // [R][long_stride] the same for the codewords of 12..16 bits, indexed by
                         //                 (16 stream bits, root bit on top) - (first[12] << 4)
    int long_stride;     //                 16 * alphabet size (more 16-bit windows cannot lie under long
                         //                 codewords), at least CO3_LONG_CACHE
    uint32_t* first;     // [R][17]         first canonical code of each length
    uint32_t* count;     // [R][17]
    uint32_t* offs;      // [R][17]         start of each length in perm
    uint8_t* perm;       // [R][256]        symbols ordered by (length, symbol)
    int32_t* ksign;      // [256]           signed integer magnitude of each symbol
};

// Bias from the current moments without a statistics pass (see co3_encode): an element whose
// a = g + gamma m cannot be rebuilt bit for bit from its symbol and its new memory is kept here.
struct Co3Side {
    uint32_t item;                // user * n_chunks + chunk
    uint32_t pos;                 // element within the chunk's tile
    uint32_t a_bits;
    uint32_t pad_;
};
constexpr int CO3_SIDE_CAP = 65536;

// Everything the kernels need, passed by value.
struct Co3Dev {
    int E, M, nm, nsym, J, cF, b_lo, b_hi;
    uint32_t Kmax;
    int U, S;
    int u_base, u_count;          // users covered by a statistics / convert launch (whole plan: 0, U)
    int64_t d, ld, sld, n_chunks, n_sub, n_groups, cap_words;
    float gamma;
    const Co3Chunk* chunks;       // [n_chunks]
    const Co3Group* groups;       // [n_groups]
    const int32_t* dec_part;      // [dec_blocks + 1] decoder: block b takes the groups (U <= 8) or chunks (U > 8)
    int dec_blocks;               //     dec_part[b] .. dec_part[b+1] - 1; a partition balanced on the host
    const int64_t* seg_off;       // [S+1]
    const int32_t* seg_chunk0;    // [S+1] first chunk of each segment
    uint8_t* sym;                 // [U][sld] internal symbols (co3_sym_internal)
    unsigned long long* hist;     // [hist_copies][S][256] by internal symbol (+ one word: the item ticket)
    int hist_copies;              // the copies are summed when the histogram is read out
    unsigned int* ticket;         // item ticket of the convert / stats pass (last word of hist)
    double* part_s1;              // [U*n_chunks] per-(user,chunk) partial sums of |a|
    double* part_s2;              //              ... of a^2
    uint32_t* part_nf;            //              ... count of non-finite a
    double* fit;                  // [S][5] beta, alpha, N, S1, S2
    int red_k;                    // > 0: the partials of a segment are first summed in red_k slices by
    double* red_s1;               //      fit_reduce_kernel ([S][red_k] each) -- plans with very long segments
    double* red_s2;
    unsigned long long* red_nf;
    int32_t* spec;                // [4] layers to convert again | blocks done | side entries | side list overflowed
    int32_t* redo_seg;            // [S] the layers whose bias turned out different from the guess ...
    int32_t* redo_old;            // [S] ... and the guess they were converted with
    Co3Side* side;                // [CO3_SIDE_CAP]
    int32_t* bias_cur;            // [S] bias used by the next convert pass
    int bias_rule;                // CO3_RULE_POLY or CO3_RULE_OPT
    const int16_t* bias_opt_tab;  // [NIBETA][8] best ir per (shape index, round(8 log2 alpha) mod 8)
    co3_seg_header* hdr_cur;      // [S] fully lagged code: header of the coming iteration (else unused)
    uint32_t* slot_buf;           // [U*n_chunks][32][CO3_SUB_WORDS] fully lagged code: the packed sub-chunks,
                                  //     each from bit 0 of its own slot, before their offsets are known (else null)
    const uint32_t* wtab;         // [NIBETA][NIR][J] model weights of the non-negative magnitudes
    const double* logr_tab;       // [2][FIT_GRID + 1] log R(beta), log G(beta) at log2(beta) uniform in [log2 0.3, 1]
    Co3CodeBook cb;               // code tables the kernels use: of all model rows, or (empirical code,
                                  // code_by_segment = 1) one row per segment, rebuilt every iteration
    int code_by_segment;
    uint32_t* chunk_words;        // [U][n_chunks] payload words of each chunk (multiple of 4)   } fully lagged
    uint32_t* chunk_bits;         // [U][n_chunks] code bits of each chunk                        } code only
    uint32_t* user_ovf;           // [U] 1 if the user's payload exceeds cap_words
    unsigned long long* enc_grp;  // [U][n_grp] single-pass encode, per group of 64 chunks: arrivals << 56 | words << 32 | bits
    uint32_t* enc_st;             // [U][n_chunks] ... published word count of each chunk (top bit: valid)
    unsigned int* enc_ticket;     // ... item ticket (the three live in one allocation, cleared per launch)
    int64_t n_grp;
    size_t enc_sync_words64;      // size of that allocation in 64-bit words
    int spin_limit;               // polls after which a wait between thread blocks gives up (CO3_FLAG_TIMEOUT)
    uint32_t* flags;              // sticky status flags
    unsigned long long* nonfinite_total;
};

struct co3_plan {
    co3_config cfg;
    Co3Dev dev;
    int64_t iteration;
    int64_t worst_case_words;
    int device;
    int num_sms;
    void* book;                     // the shared code tables of (device, format) this plan holds a reference to
    Co3CodeBook cb_emp;             // empirical-histogram code: S rows (else unallocated)
    uint8_t* emp_lens;              // ... the caller's length table during co3_encode_empirical
    const uint8_t* emp_lens_in;     // ... and during co3_decode_aggregate_empirical
    size_t enc_sync_bytes;          // size of the enc_grp / enc_st / enc_ticket allocation
    int grid_convert;               // launch grid of the convert pass (fixed per plan)
    int grid_convert_spec;          // ... of its variant that checks the guess (current-moments bias, t >= 1)
    bool two_pass_current;          // current-moments bias with a statistics pass in every iteration (CO3_TWO_PASS=1)
    cudaStream_t last_stream;
    // co3_iteration_host: copy streams and the events that order them against the caller's stream
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_h2d, ev_conv, ev_dec, ev_d2h;
    bool host_pipe_ready;           // streams and events exist
    bool ev_conv_recorded;          // a convert pass that read d_grad has been recorded
    int tiled_state;                // co3_tiled_*: 0 idle, 1 begun, 2 statistics tiles seen, 3 convert tiles seen
    int tiled_users;                // users converted so far in this tiled iteration
    float* tiled_residual;          // the residual array of its convert calls (the re-conversion in co3_tiled_finish needs it)
    double* ext_mom;                // [S][3] moments handed in by co3_moments_import
    bool use_ext_mom;               // ... and not yet consumed by a fit
    double* mom_out;                // co3_moments_export: where the reduction-only fit launch writes
    double* fit_ovr;                // [S][2] (beta, alpha) handed in by co3_set_fit_override
    bool use_fit_ovr;               // ... and in force until it is cleared
    bool record_conv;               // co3_encode records ev_conv after its last pass over the gradient
    void* allocs[128];
    int n_allocs;
    int64_t* h_seg_off;
    // tracing
    uint32_t prof_mask;
    int prof_cap;
    int prof_n[CO3_NUM_KERNELS];
    int prof_every;               // only every prof_every-th launch of a class is timed (>= 1)
    int64_t prof_seen[CO3_NUM_KERNELS];
    bool prof_open[CO3_NUM_KERNELS];
    cudaEvent_t* prof_ev;         // [CO3_NUM_KERNELS][prof_cap][2]
    int64_t launches;
};

// Event pair around the launches of kernel class k (no-ops unless the class is being traced).
inline void co3_prof_begin(co3_plan* pl, int k, cudaStream_t st) {
    pl->prof_open[k] = false;
    if ((pl->prof_mask >> k) & 1u) {
        const int every = pl->prof_every > 1 ? pl->prof_every : 1;
        if (pl->prof_seen[k]++ % every == 0 && pl->prof_n[k] < pl->prof_cap) {
            cudaEventRecord(pl->prof_ev[((size_t)k * pl->prof_cap + pl->prof_n[k]) * 2], st);
            pl->prof_open[k] = true;
        }
    }
}
inline void co3_prof_end(co3_plan* pl, int k, cudaStream_t st, int n_launches) {
    pl->launches += n_launches;
    if (pl->prof_open[k]) {
        cudaEventRecord(pl->prof_ev[((size_t)k * pl->prof_cap + pl->prof_n[k]) * 2 + 1], st);
        pl->prof_n[k]++;
        pl->prof_open[k] = false;
    }
}

// host-side helpers (co3_model.cu)
int co3_host_fmt_ok(co3_format f);
int co3_host_cF(int E, int M);
int64_t co3_host_K(int M, int j);
const uint32_t* co3_host_weight_table(int E, int M);   // [NIBETA][NIR][J], cached per format
const double* co3_host_logr_table(void);               // [2][FIT_GRID + 1], cached
const int16_t* co3_host_bias_opt_table(int E, int M);   // [NIBETA][8], cached per format

// kernel launchers (each returns a cudaError_t from the launch)
cudaError_t co3_launch_stats(co3_plan* pl, const float* g, const float* m, int u_base, int u_count, cudaStream_t st);
cudaError_t co3_launch_convert(co3_plan* pl, const float* g, float* m, int u_base, int u_count, bool first,
                               cudaStream_t st, bool cleared = false, bool check_guess = false);
cudaError_t co3_launch_reconvert(co3_plan* pl, float* m, cudaStream_t st);
cudaError_t co3_launch_convert_pack(co3_plan* pl, const float* g, float* m, uint16_t* sub_bits, cudaStream_t st);
cudaError_t co3_launch_scan_gather(co3_plan* pl, uint32_t* bitstream, const uint16_t* sub_bits, uint32_t* chunk_off,
                                   unsigned long long* user_bits, cudaStream_t st);
cudaError_t co3_launch_fit(co3_plan* pl, int mode, co3_seg_header* hdr, cudaStream_t st, bool clear_hist = false,
                           float* residual = nullptr);   // residual: mode 6 only
cudaError_t co3_build_codebook(co3_plan* pl, cudaStream_t st);
// empirical-histogram code: S codes from this iteration's histogram (lengths also to code_lens, device
// [S][2^B]), or the tables of the codes whose lengths are given
cudaError_t co3_build_hist_codes(co3_plan* pl, uint8_t* code_lens, cudaStream_t st);
cudaError_t co3_build_codes_from_lens(co3_plan* pl, const uint8_t* code_lens, cudaStream_t st);
cudaError_t co3_launch_encode(co3_plan* pl, const co3_seg_header* hdr, uint32_t* bitstream,
                              uint16_t* sub_bits, uint32_t* chunk_off, unsigned long long* user_bits,
                              cudaStream_t st);
cudaError_t co3_launch_decode(co3_plan* pl, const uint32_t* bitstream, const uint16_t* sub_bits,
                              const uint32_t* chunk_off, const co3_seg_header* hdr, float* avg,
                              float* weights, float step, cudaStream_t st);
cudaError_t co3_launch_encode_stalled(co3_plan* pl, const co3_seg_header* hdr, uint32_t* bitstream,
                                      uint16_t* sub_bits, uint32_t* chunk_off, unsigned long long* user_bits,
                                      int spin_limit, cudaStream_t st);
// Decoder work split (host): fills part[0 .. n_blocks] for at most max_blocks blocks, returns n_blocks.
// teams: teams per block of the decoder that will run; items are groups (U <= 8) or chunks (U > 8).
int co3_decode_partition(const Co3Chunk* chunks, int64_t n_chunks, const Co3Group* groups, int64_t n_groups, int U,
                         int max_blocks, int32_t* part);
int co3_decode_max_blocks(int U, int num_sms);
int co3_host_balanced_split(const double* w, const int32_t* seg, int64_t n, int teams, int max_blocks, double run_cost,
                            int32_t* part);
cudaError_t co3_setup_kernels(void);
cudaError_t co3_launch_symbol_export(co3_plan* pl, uint8_t* symbols, cudaStream_t st);

// Model row of a segment header; out-of-range indices (a corrupt header) are clamped and reported.
__host__ __device__ inline int co3_row_of(const co3_seg_header h, bool* bad) {
    int ib = (int)h.ibeta, ir = (int)h.ir;
    if (ib < CO3_IBETA_MIN || ib > CO3_IBETA_MAX || ir < CO3_IR_MIN || ir > CO3_IR_MAX) {
        *bad = true;
        ib = ib < CO3_IBETA_MIN ? CO3_IBETA_MIN : (ib > CO3_IBETA_MAX ? CO3_IBETA_MAX : ib);
        ir = ir < CO3_IR_MIN ? CO3_IR_MIN : (ir > CO3_IR_MAX ? CO3_IR_MAX : ir);
    }
    return (ib - CO3_IBETA_MIN) * CO3_NIR + (ir - CO3_IR_MIN);
}

// Inside the library a symbol is stored as (magnitude code << 1) | sign instead of the public
// sign << (E+M) | magnitude code: the frequent symbols (small and medium magnitudes of both
// signs) are then neighbours, so table look-ups of a warp spread over distinct shared-memory banks.
__host__ __device__ inline int co3_sym_internal(int sym, int nm) { return ((sym & ((1 << nm) - 1)) << 1) | (sym >> nm); }
__host__ __device__ inline int co3_sym_public(int isym, int nm) { return ((isym & 1) << nm) | (isym >> 1); }

// The same from the internal symbol form (magnitude code << 1 | sign).
__host__ __device__ inline int32_t co3_ksigned_internal(int isym, int M) {
    const int j = isym >> 1, e = j >> M, f = j & ((1 << M) - 1);
    const int32_t k = (e == 0) ? f : (((1 << M) + f) << (e - 1));
    return (isym & 1) ? -k : k;
}

// Signed integer magnitude of a symbol byte: K(j) = f (e = 0) or (2^M + f) << (e - 1).
__host__ __device__ inline int32_t co3_ksigned(int sym, int M, int nm) {
    int j = sym & ((1 << nm) - 1);
    int e = j >> M, f = j & ((1 << M) - 1);
    int32_t k = (e == 0) ? f : (((1 << M) + f) << (e - 1));
    return (sym >> nm) ? -k : k;
}
