/*
 * co3.h -- C ABI of the B200 (sm_100a) CO3 gradient pipeline.
 *
 * CO3 ("convert, compress, correct") is the per-iteration gradient processing of Algorithm 1 of
 * the paper: at every user u, ghat = Q_fp(g + gamma m) (line 8), b = h_Hf(ghat) (line 9),
 * m <- gamma m + g - ghat (line 10); at the parameter server, decode every user's stream
 * (line 13) and average (line 14, Eq. "aggregate").  Q_fp is the conversion to a float with 1
 * sign, `exp_bits` exponent and `mant_bits` mantissa bits and an exponent bias b_t chosen per
 * layer from a generalized-normal fit (Sec. III (i), Eq. "exp bias", Eq. "approximate"); h_Hf is
 * an element-wise Huffman code, one per layer and shared by all users, designed from the same
 * fitted model (Sec. III (ii)).
 *
 * Conventions
 *  - Every pointer marked "device" is CUDA device memory owned by the caller; "host" is host
 *    memory.  The plan owns its scratch, tables, status word, and the two copy streams and four
 *    events of co3_iteration_host; no call after co3_plan_create allocates device memory or creates
 *    a stream or an event (co3_profile_enable creates the events it is asked for; the inspection
 *    hooks co3_debug_* use temporary host memory).
 *  - co3_encode / co3_decode_aggregate only enqueue work on `cuda_stream` (a cudaStream_t cast
 *    to void*, NULL = default stream) and return without synchronising.  Calls on one plan must
 *    be issued on one stream (or be ordered by the caller).
 *  - Return value: 0, or a negative CO3_E* code for errors detected on the host.  Conditions
 *    detected on the device (non-finite inputs, payload capacity, corrupt stream) set sticky
 *    flags read with co3_status.  Nothing throws, prints or exits.
 *  - Row layout: user u's vectors start at element u*ld of `grad` / `residual`; ld >= d,
 *    ld % 4 == 0 and the base pointers are 16-byte aligned.  A "segment" is a layer: a range
 *    [seg_offsets[l], seg_offsets[l+1]) of every user's row with its own bias and code.
 *
 * Container (what co3_encode writes and co3_decode_aggregate reads).  A row is cut into chunks
 * at every multiple of 4096 elements and at every segment boundary, and each chunk into
 * sub-chunks at every multiple of 128 elements.  Chunk c of user u is the 32-bit words
 * [chunk_off[u][c], chunk_off[u][c+1]) of bitstream row u; its word count is its bit count
 * rounded up to a multiple of 128 bits.  Codewords are packed without gaps, stream bit p is bit
 * (p & 31) of word (p >> 5), a codeword's root bit first, pad bits zero.  sub_bits[u][k] is the
 * bit length of sub-chunk k (numbered along the row).  The per-segment header (bias and the two
 * indices that name the code model) is shared by all users.
 */
#ifndef CO3_H
#define CO3_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CO3_OK 0
#define CO3_EINVAL (-1)     /* bad argument or unsupported configuration            */
#define CO3_ENOMEM (-2)     /* device or host allocation failed in co3_plan_create  */
#define CO3_ECUDA (-3)      /* a CUDA runtime call failed                            */
#define CO3_ECAPACITY (-4)  /* a user's payload does not fit cap_words               */
#define CO3_ECORRUPT (-5)   /* a stream did not decode to its recorded lengths       */
#define CO3_ENONFINITE (-6) /* NaN/Inf met in g + gamma m (coded as 0, memory reset) */
#define CO3_ELIMIT (-7)     /* input larger than the fixed scratch of co3_moments_static */

#define CO3_FLAG_CAPACITY 1u
#define CO3_FLAG_CORRUPT 2u
#define CO3_FLAG_NONFINITE 4u
#define CO3_FLAG_TIMEOUT 8u  /* a bounded wait between thread blocks ran out (should never happen) */
#define CO3_FLAG_INEXACT 16u /* CO3_BIAS_CURRENT only: in one iteration more than 65536 elements lay at least 2^(23-M)
                                times beyond the largest value that the PREVIOUS iteration's bias of their layer could
                                represent, and a layer's bias changed: some of them were converted at the previous
                                bias (see the note on CO3_BIAS_CURRENT) */

/* CO3_BIAS_CURRENT is Algorithm 1 as printed: the bias b_t is chosen "at each time t" for the
 * distribution of g_t + gamma m_{t-1} itself (Sec. III (i), Eq. "exp bias").  Taken literally that is an
 * extra read pass over gradient and memory in front of every conversion.  co3_encode runs that pass at
 * t = 0 only.  For t >= 1 it converts under the bias of iteration t-1, takes the moments of
 * g_t + gamma m_{t-1} from that same pass (the same sums in the same order), derives b_t from them, and
 * converts again -- from the stored symbol and memory, g + gamma m = q + m' exactly -- only the layers
 * whose b_t differs from the bias they were converted with.  Symbols, memory, histogram, header and
 * payload are bit for bit those of the two-pass order (the environment variable CO3_TWO_PASS=1, read
 * when a plan is made, keeps the statistics pass in every iteration; a test compares the two).  An
 * element so far beyond the format's range under the previous bias that q + m' would not give it back
 * is kept on a side list of 65536 entries and converted from there; should an iteration have more of
 * them, CO3_FLAG_INEXACT is raised.  The co3_tiled_* calls do the same (co3_tiled_finish repairs).
 * CO3_BIAS_LAGGED is NOT Algorithm 1's per-iteration bias: that pass runs at t = 0 only, and b_t for
 * t >= 1 is the rule applied to the fit of iteration t-1 (whose moments ride along with its conversion
 * pass); the code of iteration t is still designed from iteration t's own fit.  It relies on the fitted
 * model drifting slowly from one iteration to the next. */
#define CO3_BIAS_CURRENT 0
#define CO3_BIAS_LAGGED 1
/* Not in the paper's Algorithm 1, which fits "at each time t": bias AND code model of iteration
 * t >= 1 come from the fit of iteration t-1, so the whole header of an iteration is known before its
 * gradient is seen and conversion and packing are one pass over the data (the symbols never go to
 * memory).  Symbols, residuals and averages are exactly those of CO3_BIAS_LAGGED; only the code
 * differs (by one iteration), at a rate that is higher by the drift of the model per iteration.
 * co3_debug_symbols is not available in this mode. */
#define CO3_CODE_LAGGED 2
/* Not the paper's code design (which builds the code from the fitted GenNorm model): the bias is
 * handled as in CO3_BIAS_LAGGED, but the code of every layer is the Huffman code of this iteration's
 * own symbol histogram (pooled over users, same construction as the model code: full alphabet, floor
 * 1, depth at most 16), and the table of its code lengths is side information: 2^(1+E+M) bytes per
 * layer per iteration.  Use co3_encode_empirical / co3_decode_aggregate_empirical with such a plan. */
#define CO3_CODE_EMPIRICAL 3

/* How the exponent bias follows from the fitted GenNorm (Sec. III (i)).
 * CO3_RULE_POLY: the paper's closed form (Eq. "approximate"): b = nearest integer to
 *   log2(alpha) - log2(0.46 - 2.85 beta + 5.37 beta^2 - 2.85 beta^3 + 0.52 beta^4), fitted by the
 *   paper for its 4-bit format.
 * CO3_RULE_OPT: what that closed form approximates (Eq. "exp bias", L2 reading), for the plan's own
 *   format: the integer b that minimises the expected squared conversion error of the fitted
 *   GenNorm, evaluated on the header grid (shape 2^(ibeta/8), log2(alpha) - b in steps of 1/8). */
#define CO3_RULE_POLY 0
#define CO3_RULE_OPT 1

typedef struct co3_plan co3_plan; /* opaque, library-owned */

/* Sec. III (i): one sign bit is implied.  Supported: 1 <= exp_bits <= 4, 1 <= mant_bits,
 * exp_bits + mant_bits <= 7; (4,3), (3,2) and (1,2) are the 8-, 6- and 4-bit formats. */
typedef struct {
    int32_t exp_bits, mant_bits;
} co3_format;

/* What the parameter server needs per segment to rebuild grid and code: the integer exponent
 * bias b (grid value = +-K(j) * 2^(b + 1 - bias_F - mant_bits)), and the fitted GenNorm shape
 * and scale on a 1/8-octave grid: beta_q = 2^(ibeta/8), alpha_q = 2^(b + ir/8). */
typedef struct {
    int8_t bias;
    int8_t ibeta;
    int16_t ir;
} co3_seg_header;

typedef struct {
    int64_t d;                  /* elements per user                                              */
    int64_t ld;                 /* row pitch of grad/residual in elements, >= d, multiple of 4    */
    int32_t n_users;            /* U; n_users * K_max < 2^24 (K_max: largest integer magnitude)    */
    co3_format fmt;
    int32_t n_segments;         /* S >= 1                                                          */
    const int64_t* seg_offsets; /* host, S+1 non-decreasing entries, [0] = 0, [S] = d; NULL: S = 1 */
    float gamma;                /* memory decay of Algorithm 1 line 8; 0: no feedback, 1: plain EF */
    int32_t bias_mode;          /* CO3_BIAS_CURRENT, CO3_BIAS_LAGGED, CO3_CODE_LAGGED, CO3_CODE_EMPIRICAL */
    int64_t cap_words;          /* row pitch of `bitstream` in 32-bit words, multiple of 4         */
    int32_t bias_rule;          /* CO3_RULE_POLY (the paper's, default 0) or CO3_RULE_OPT          */
    int32_t reserved;           /* 0                                                               */
} co3_config;

/* Algorithm 1 line 2 and Table I: fixes d, U, the format, the layers, gamma.  Validates the
 * configuration, computes the static chunk partition, builds the GenNorm model-weight table on
 * the host, allocates all device scratch on the current device and builds there the Huffman code
 * (Sec. III (ii)) of every (shape, scale) pair a header can name, so that an iteration only selects
 * codes.  Those code tables depend on the format alone: the plans of one device and format share one
 * copy, built by the first of them and freed with the last (plan creation and destruction take a
 * process-wide lock for that).  The iteration counter
 * starts at 0 (memory m_0 = 0 is the caller's zero-filled `residual`).
 * Every call that takes a stream only enqueues work on it (kernels, memsets, device-to-device copies)
 * and never waits for the device, so a steady-state iteration (t >= 1 with CO3_BIAS_LAGGED or
 * CO3_CODE_LAGGED or CO3_BIAS_CURRENT; tracing off) may be recorded by stream capture and
 * replayed as a CUDA graph: the kernel sequence does not depend on t.  Iteration 0
 * runs an extra statistics pass and must be run, not replayed, first.  (The iteration counter that
 * co3_state_export reports counts calls, not replays of a graph that recorded one.) */
int co3_plan_create(co3_plan** out, const co3_config* cfg);
void co3_plan_destroy(co3_plan* plan);

/* Sizes of the side-information arrays and the worst-case payload (16 bits per symbol plus
 * chunk padding) in words per user.  Any pointer may be NULL. */
int co3_sizes(const co3_plan* plan, int64_t* n_chunks, int64_t* n_sub, int64_t* worst_case_words);

/* Algorithm 1 lines 8-10 for all users (one iteration t, then t <- t + 1):
 *   grad      device, const, [U][ld] fp32   g_t^(u)
 *   residual  device, in/out, [U][ld] fp32  m_{t-1}^(u) -> m_t^(u)
 *   bitstream device, out, [U][cap_words]   h_Hf(ghat_t^(u)), container as described above
 *   sub_bits  device, out, [U][n_sub] u16
 *   chunk_off device, out, [U][n_chunks+1] u32, in words
 *   user_bits device, out, [U] u64          r_t^(u): code bits of user u
 *   hdr       device, out, [n_segments]
 * If a user's payload would exceed cap_words, CO3_FLAG_CAPACITY is raised; nothing is written at
 * or beyond cap_words of a row, the chunks that would not fit are not written, and the row's
 * content is then unspecified; chunk_off, sub_bits and user_bits are still written in full.
 * Non-finite g + gamma m: counted, coded as +0, memory reset to 0, CO3_FLAG_NONFINITE raised. */
int co3_encode(co3_plan* plan, const float* grad, float* residual, uint32_t* bitstream,
               uint16_t* sub_bits, uint32_t* chunk_off, uint64_t* user_bits, co3_seg_header* hdr,
               void* cuda_stream);

/* The same iteration fed in tiles of users, for gradients of all users that do not fit the device
 * at once (residual, payload and side information still cover all users and stay resident; only the
 * gradient buffer holds a tile and is refilled by the caller between calls):
 *   co3_tiled_begin       starts the iteration; *need_statistics = 1 if the bias has to come from a
 *                         statistics pass first (t = 0; with CO3_BIAS_CURRENT and CO3_TWO_PASS=1 every t)
 *   co3_tiled_statistics  (only then) once for every tile: grad_tile is [n_tile_users][ld] for the
 *                         users user0 .. user0 + n_tile_users - 1, residual the full [U][ld] array
 *   co3_tiled_convert     once for every tile, after all statistics calls: as co3_encode's convert
 *                         step for those users
 *   co3_tiled_finish      fit, header, coding of all users; the iteration counter advances
 * Every user must be covered exactly once per pass; the result is bit for bit that of co3_encode.
 * Not available with CO3_CODE_LAGGED and CO3_CODE_EMPIRICAL plans. */
int co3_tiled_begin(co3_plan* plan, int32_t* need_statistics);
int co3_tiled_statistics(co3_plan* plan, const float* grad_tile, const float* residual, int32_t user0,
                         int32_t n_tile_users, void* cuda_stream);
int co3_tiled_convert(co3_plan* plan, const float* grad_tile, float* residual, int32_t user0,
                      int32_t n_tile_users, void* cuda_stream);
int co3_tiled_finish(co3_plan* plan, uint32_t* bitstream, uint16_t* sub_bits, uint32_t* chunk_off,
                     uint64_t* user_bits, co3_seg_header* hdr, void* cuda_stream);

/* Pooled moments across plans (a gradient cut into slices of d, one plan per slice, e.g. one per GPU).
 * The shape and scale of a layer are fitted to the moments of ALL its entries (Sec. III (i), the
 * moment-matching fit), so a layer that spans several slices needs its three sums added over the
 * slices before the fit; everything else of an iteration is local to a slice.  Inside a tiled
 * iteration, after the last co3_tiled_statistics call and again after the last co3_tiled_convert call:
 *   co3_moments_export  moments: device, out, [n_segments][3] fp64 = (finite entries, sum |a|, sum a^2)
 *                       of this plan's part of every segment, a = g + gamma m, all users pooled
 *   co3_moments_import  moments: device, const, same layout: the sums the next fit (the bias before the
 *                       first convert tile, or the header in co3_tiled_finish) uses INSTEAD of the
 *                       plan's own; consumed by that fit.  The caller adds the exported sums of the
 *                       plans that share a segment (an all-reduce of n_segments x 3 doubles) in between.
 * Without an import the plan's own sums are used, as before.  CO3_EINVAL outside those two places. */
int co3_moments_export(co3_plan* plan, double* moments, void* cuda_stream);
int co3_moments_import(co3_plan* plan, const double* moments, void* cuda_stream);

/* Algorithm 1 lines 13-14 without the model update: decode all U streams and write
 * avg_grad[i] = (1/U) sum_u ghat^(u)[i] (Eq. "aggregate"), device [d] fp32.  Depends only on
 * its arguments and the plan's static configuration, never on encoder scratch.  The integer
 * magnitudes are summed exactly and scaled once, so the result does not depend on the order of
 * the users.  A stream that does not decode to its recorded lengths raises CO3_FLAG_CORRUPT;
 * no out-of-bounds access is made for any input bytes. */
int co3_decode_aggregate(co3_plan* plan, const uint32_t* bitstream, const uint16_t* sub_bits,
                         const uint32_t* chunk_off, const co3_seg_header* hdr, float* avg_grad,
                         void* cuda_stream);

/* The two calls for a CO3_CODE_EMPIRICAL plan (the others return CO3_EINVAL for it, and these for any
 * other plan).  code_lens: device, [n_segments][2^(1+E+M)] u8, the code length of every symbol byte:
 * written by the encoder, read by the decoder, which rebuilds the canonical codes from it and raises
 * CO3_FLAG_CORRUPT if the lengths are not those of a complete prefix code of depth <= 16.  hdr is
 * still written and read (the decoder needs the bias; the model indices are informational). */
int co3_encode_empirical(co3_plan* plan, const float* grad, float* residual, uint32_t* bitstream,
                         uint16_t* sub_bits, uint32_t* chunk_off, uint64_t* user_bits, co3_seg_header* hdr,
                         uint8_t* code_lens, void* cuda_stream);
int co3_decode_aggregate_empirical(co3_plan* plan, const uint32_t* bitstream, const uint16_t* sub_bits,
                                   const uint32_t* chunk_off, const co3_seg_header* hdr,
                                   const uint8_t* code_lens, float* avg_grad, void* cuda_stream);

/* The same with the model update of Algorithm 1 line 14 fused in: besides avg_grad,
 * weights[i] <- fl32(weights[i] + fl32(step * avg_grad[i])) (device, in/out, [d] fp32; two roundings,
 * no fused multiply-add).  The paper writes the update with both signs (Sec. II, Algorithm 1), so
 * the caller passes the signed step: -eta for descent. */
int co3_decode_aggregate_update(co3_plan* plan, const uint32_t* bitstream, const uint16_t* sub_bits,
                                const uint32_t* chunk_off, const co3_seg_header* hdr, float* avg_grad,
                                float* weights, float step, void* cuda_stream);

/* One whole iteration from host memory (what a training loop that keeps gradients on the host
 * would call): copies h_grad (host, [U][ld], pinned for full speed) to d_grad, runs co3_encode
 * and co3_decode_aggregate with the given device buffers, and copies the average back to h_avg
 * (host, [d]).  The caller synchronises cuda_stream, as for the other calls: the two copies run on
 * streams of the plan, ordered against cuda_stream with events, so that the gradient copy of the next
 * call overlaps this call's encode, decode and copy back.  d_grad is scratch of this call sequence:
 * nothing else may touch it between calls, and h_grad may be reused once cuda_stream has been
 * synchronised (or the next call's work on it has completed). */
int co3_iteration_host(co3_plan* plan, const float* h_grad, float* d_grad, float* d_residual,
                       uint32_t* d_bitstream, uint16_t* d_sub_bits, uint32_t* d_chunk_off,
                       uint64_t* d_user_bits, co3_seg_header* d_hdr, float* d_avg, float* h_avg,
                       void* cuda_stream);

/* Synchronises the stream last used by the plan and reports the sticky flags and the running
 * count of non-finite inputs.  clear != 0 resets both.  Returns CO3_OK or CO3_ECUDA. */
int co3_status(co3_plan* plan, uint32_t* flags, uint64_t* nonfinite_count, int32_t clear);

/* Fit of the last encoded iteration for one segment (synchronises): GenNorm shape and scale by
 * moment matching, and the pooled moments N, sum|a|, sum a^2 of a = g + gamma m. */
int co3_get_fit(co3_plan* plan, int32_t seg, double* beta, double* alpha, double* N, double* S1,
                double* S2);

/* Checkpoint/resume of what the method carries between iterations besides the caller's
 * residual: the iteration counter and the next bias per segment (host int32 [n_segments]).
 * With CO3_CODE_LAGGED the next header is carried too: co3_state_header copies it out of
 * (import == 0) or into (import != 0) the plan, host [n_segments]. */
int co3_state_export(co3_plan* plan, int64_t* iteration, int32_t* next_bias);
int co3_state_import(co3_plan* plan, int64_t iteration, const int32_t* next_bias);
int co3_state_header(co3_plan* plan, int32_t import, co3_seg_header* next_header);

/* Tracing: per-kernel device time measured with CUDA events recorded on the caller's stream
 * around the launches of the selected kernel classes.  co3_profile_enable creates the events
 * (max_records launches per class between two collects; mask 0 frees them);
 * co3_profile_collect synchronises, adds up the recorded launches of each class since the last
 * collect (total_ms and launches are host arrays of CO3_NUM_KERNELS entries) and starts over.
 * co3_launch_count: number of the library's kernels launched on this plan so far. */
#define CO3_K_STATS 0        /* moments of g + gamma m (t = 0, or every t in CURRENT mode) */
#define CO3_K_FIT 1          /* GenNorm fit, bias, header                                   */
#define CO3_K_CONVERT 2      /* fused EF-add / convert / residual / histogram / moments      */
#define CO3_K_CODE_ENC 3     /* CO3_CODE_EMPIRICAL only: code build from the histogram (model codes are built once, at plan creation) */
#define CO3_K_RECONVERT 4    /* CO3_BIAS_CURRENT, t >= 1: layers whose bias differs from the guess, converted again */
#define CO3_K_ENC_SCAN 5     /* chunk offsets (CO3_CODE_LAGGED only)                         */
#define CO3_K_ENC_PACK 6     /* lengths + offsets + bit packing (CO3_CODE_LAGGED: concatenation) */
#define CO3_K_CODE_DEC 7     /* CO3_CODE_EMPIRICAL only: decoder tables from the received code lengths */
#define CO3_K_DECODE 8       /* decode + aggregate                                           */
#define CO3_NUM_KERNELS 9
int co3_profile_enable(co3_plan* plan, uint32_t kernel_mask, int32_t max_records);
int co3_profile_collect(co3_plan* plan, double* total_ms, int64_t* launches);
/* Time only every `every`-th launch of each traced class (default 1: all of them): two event records
 * cost about as much device time as a small kernel, so a long timed loop may want to sample.
 * co3_profile_collect then reports the sampled launches and their total. */
int co3_profile_stride(co3_plan* plan, int32_t every);
int64_t co3_launch_count(const co3_plan* plan);

/* Inspection hooks (synchronise; used by the parity tests).
 * symbols: device out [U][d] u8, the converted symbols of the last iteration
 *          (sign << (E+M) | exponent << M | mantissa).
 * hist:    host out [n_segments][2^(1+E+M)] u64, symbol counts pooled over users.
 * code:    host out, lengths [n_segments][2^B] u8 and codewords [n_segments][2^B] u32 (root bit
 *          = most significant of `length` bits) of the codes that the headers `hdr` (device,
 *          [n_segments]) select. */
int co3_debug_symbols(co3_plan* plan, uint8_t* symbols, void* cuda_stream);
int co3_debug_hist(co3_plan* plan, uint64_t* hist);
int co3_debug_code(co3_plan* plan, const co3_seg_header* hdr, uint8_t* lengths, uint32_t* codewords);

/* Test hook: from now on every fit of this plan takes (beta, alpha) of segment l from fit[2l], fit[2l+1]
 * (host, [n_segments][2]; alpha = 0 means the degenerate all-zero segment) instead of solving the moment
 * equations; bias and header follow from them by the usual rules, the moments reported by co3_get_fit
 * stay the plan's own.  NULL switches it off.  A harness uses it to feed another implementation's fit
 * and so tell a header that differs by a rounding of the fit from a fault further down.  Synchronises. */
int co3_set_fit_override(co3_plan* plan, const double* fit);

/* Test hook for the bounded waits of the encoder.  The thread blocks of co3_encode's packing kernel
 * learn their chunk's place from the sizes that the blocks of the earlier chunks publish; each such wait
 * polls a limited number of times and then gives up, raises CO3_FLAG_TIMEOUT and writes no payload.
 * This call runs that kernel over the symbols of the last co3_encode with the block of (user 0, chunk 0)
 * left out and the limit set to spin_limit polls (1 .. 2^20), so that the waits for that chunk's size run
 * out: afterwards co3_status reports CO3_FLAG_TIMEOUT, the chunks of user 0 after the first are not
 * written, and the device is as usable as before.  Needs a plan that keeps symbols (not
 * CO3_CODE_LAGGED, not CO3_CODE_EMPIRICAL), at least one encoded iteration and at least two chunks. */
int co3_debug_encode_stalled(co3_plan* plan, uint32_t* bitstream, uint16_t* sub_bits, uint32_t* chunk_off,
                             uint64_t* user_bits, const co3_seg_header* hdr, int32_t spin_limit,
                             void* cuda_stream);

/* Host only, no GPU needed: integer model weights of the quantised GenNorm source for header
 * indices (ibeta in [-14, 8], ir in [-96, 31]), one per symbol byte, 2^(1+E+M) entries.  The
 * Huffman code of a segment is built from exactly these numbers (Sec. III (ii)). */
int co3_model_weights(co3_format fmt, int32_t ibeta, int32_t ir, uint32_t* weights);

/* Host only.  Users and parameter server rebuild every code from the header alone (Algorithm 1 lines 9
 * and 13), i.e. from these weights, which each side computes with its own math library (lgamma, pow,
 * exp): the two sides agree when they run the same build of this library against the same libm.  This
 * is a 64-bit FNV-1a digest of the whole weight table of a format (all 23 x 128 index pairs); exchange
 * and compare it once before the first iteration.  0: unsupported format or out of memory. */
uint64_t co3_model_checksum(co3_format fmt);

/* Host only: the table behind CO3_RULE_OPT, 23 x 8 int16: for shape index ibeta + 14 and residue
 * rho = round(8 log2 alpha) mod 8, the ir (congruent to rho) of least expected squared conversion
 * error; the rule's bias is (round(8 log2 alpha) - ir) / 8, clamped.  co3_grid_distortion is the
 * objective itself, E[(Q(X) - X)^2] / alpha^2 at a header cell (negative: invalid arguments). */
int co3_bias_opt_table(co3_format fmt, int16_t* table);
double co3_grid_distortion(co3_format fmt, int32_t ibeta, int32_t ir);

/* Host only: the static partition for (d, segments), as co3_plan_create computes it.  Arrays
 * are host, sized by a first call with NULL arrays that returns the chunk count. */
int64_t co3_partition(int64_t d, int32_t n_segments, const int64_t* seg_offsets,
                      int32_t* chunk_seg, int64_t* chunk_start, int64_t* chunk_end,
                      int64_t* sub_base, int64_t* n_sub);

/* Host only: how co3_plan_create splits the work of the multi-user decoders over their thread blocks.
 * n items in order, each with a cost (host, double; 1 = a full chunk) and a segment number (host, int32);
 * a block takes a contiguous range and walks it run by run of one segment, its `teams` (1..32) teams
 * taking every teams-th item of a run and meeting where the segment changes.  The time of a run is
 * modelled as the mean of the cost of its most loaded team and of its total cost / teams (what binds
 * when all teams are busy), plus a fixed 0.04 for the change of code tables; a block takes the sum over
 * its runs.  part (host, max_blocks + 1 entries) receives cuts whose largest block time is the least
 * that a contiguous split into at most max_blocks blocks reaches, with the work spread over all
 * min(max_blocks, n) blocks in proportion within that bound: block b takes items part[b] .. part[b+1] - 1.
 * Returns the number of blocks in use, or a negative value for bad arguments. */
int co3_balanced_split(const double* cost, const int32_t* seg, int64_t n, int32_t teams, int32_t max_blocks,
                       int32_t* part);

/* (The paper has no counterpart of this call: it is a convenience of this library.)
 * Pooled moments of a = g + gamma m over n elements, WITHOUT allocating anything: for callers
 * that may not allocate device memory when they need these statistics -- code living inside a
 * host application whose device memory belongs to that application's own pool, or loops that
 * cannot take the device-wide synchronisation of cudaMalloc/cudaFree -- and that therefore cannot
 * create a plan (co3_plan_create allocates tables and scratch).
 *   grad, residual  device, const, n fp32 each, 16-byte aligned (for several users pass the
 *                   rows back to back: n = U * d with ld == d)
 *   moments         device, out, 4 doubles: N (finite elements), sum |a|, sum a^2, non-finite count
 * The partial sums live in a 3 MiB array that is part of the library's device image (every GPU
 * that loads the library holds it until the process exits); n may be at most
 * CO3_STATIC_MAX_ELEMENTS, else CO3_ELIMIT is returned and nothing is launched.  The first call
 * on each device looks the array's device address up: make it before any stream capture begins.
 * All calls share the array, so calls whose kernels could overlap on the GPU (other streams,
 * other host threads) must be serialised by the caller; nothing in it needs clearing between
 * calls.  Work is enqueued on cuda_stream; the caller synchronises before reading `moments`. */
#define CO3_STATIC_MAX_ELEMENTS ((int64_t)1 << 29)
int co3_moments_static(const float* grad, const float* residual, int64_t n, float gamma,
                       double* moments, void* cuda_stream);

const char* co3_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CO3_H */
