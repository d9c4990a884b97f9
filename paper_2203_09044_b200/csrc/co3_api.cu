// C ABI of the CO3 library: plan management and the kernel sequences of one iteration of
// Algorithm 1 (lines 8-10 at the users: co3_encode; lines 13-14 at the server:
// co3_decode_aggregate).  Everything is enqueued on the caller's stream; nothing here allocates
// after co3_plan_create and nothing synchronises except the inspection calls.
#include <mutex>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "co3_internal.h"

cudaError_t co3_setup_decode_kernels(void);

namespace {

template <typename T>
int dev_alloc(co3_plan* pl, T** out, size_t count) {
    void* ptr = nullptr;
    if (pl->n_allocs >= 64) return CO3_ENOMEM;
    if (cudaMalloc(&ptr, (count ? count : 1) * sizeof(T)) != cudaSuccess) {
        (void)cudaGetLastError();
        return CO3_ENOMEM;
    }
    pl->allocs[pl->n_allocs++] = ptr;
    *out = (T*)ptr;
    return CO3_OK;
}

int alloc_codebook(co3_plan* pl, Co3CodeBook& cb, size_t R, int ncand) {
    int rc = 0;
    cb.ncand = ncand;
    rc |= dev_alloc(pl, &cb.cand_len, R * (size_t)ncand * CO3_MAXSYM);
    rc |= dev_alloc(pl, &cb.cand_max, R * (size_t)ncand);
    rc |= dev_alloc(pl, &cb.len8, R * CO3_MAXSYM);
    rc |= dev_alloc(pl, &cb.len_pub, R * CO3_MAXSYM);
    rc |= dev_alloc(pl, &cb.enc, R * CO3_MAXSYM);
    rc |= dev_alloc(pl, &cb.code_msb, R * CO3_MAXSYM);
    rc |= dev_alloc(pl, &cb.lut, R * CO3_LUT_SIZE);
    cb.long_stride = 16 * pl->dev.nsym < CO3_LONG_CACHE ? CO3_LONG_CACHE : 16 * pl->dev.nsym;
    rc |= dev_alloc(pl, &cb.lut_long, R * (size_t)cb.long_stride);
    rc |= dev_alloc(pl, &cb.first, R * (CO3_MAXLEN + 1));
    rc |= dev_alloc(pl, &cb.count, R * (CO3_MAXLEN + 1));
    rc |= dev_alloc(pl, &cb.offs, R * (CO3_MAXLEN + 1));
    rc |= dev_alloc(pl, &cb.perm, R * CO3_MAXSYM);
    rc |= dev_alloc(pl, &cb.ksign, (size_t)CO3_MAXSYM);
    return rc ? CO3_ENOMEM : CO3_OK;
}

inline cudaStream_t as_stream(void* s) { return (cudaStream_t)s; }

// The code tables of all model rows are a pure function of the format (148 MB for E4M3), so the plans
// of one device and format share one copy: built by the first plan, freed with the last.
struct SharedBook {
    int device, E, M, refs;
    Co3CodeBook cb;
    void* allocs[16];
    int n_allocs;
};
constexpr int MAX_BOOKS = 32;
SharedBook g_books[MAX_BOOKS];
std::mutex g_books_mutex;

template <typename T>
bool book_alloc(SharedBook& b, T** out, size_t count) {
    void* ptr = nullptr;
    if (b.n_allocs >= 16 || cudaMalloc(&ptr, (count ? count : 1) * sizeof(T)) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    b.allocs[b.n_allocs++] = ptr;
    *out = (T*)ptr;
    return true;
}

void book_free(SharedBook& b) {
    for (int i = 0; i < b.n_allocs; ++i) cudaFree(b.allocs[i]);
    b = SharedBook{};
}

// Takes a reference to the book of (pl->device, format), building it with the plan's own configuration
// if it does not exist yet (the plan's static tables must already be on the device).
int book_acquire(co3_plan* pl) {
    std::lock_guard<std::mutex> lock(g_books_mutex);
    const int E = pl->dev.E, M = pl->dev.M;
    SharedBook* slot = nullptr;
    for (SharedBook& b : g_books) {
        if (b.refs > 0 && b.device == pl->device && b.E == E && b.M == M) {
            ++b.refs;
            pl->dev.cb = b.cb;
            pl->book = &b;
            return CO3_OK;
        }
        if (b.refs == 0 && !slot) slot = &b;
    }
    if (!slot) return CO3_ENOMEM;
    SharedBook& b = *slot;
    b = SharedBook{};
    Co3CodeBook& cb = b.cb;
    const size_t R = CO3_NROWS;
    cb.ncand = CO3_NCAND;
    cb.long_stride = 16 * pl->dev.nsym < CO3_LONG_CACHE ? CO3_LONG_CACHE : 16 * pl->dev.nsym;
    bool ok = book_alloc(b, &cb.cand_len, R * (size_t)cb.ncand * CO3_MAXSYM) && book_alloc(b, &cb.cand_max, R * (size_t)cb.ncand) &&
              book_alloc(b, &cb.len8, R * CO3_MAXSYM) && book_alloc(b, &cb.len_pub, R * CO3_MAXSYM) &&
              book_alloc(b, &cb.enc, R * CO3_MAXSYM) && book_alloc(b, &cb.code_msb, R * CO3_MAXSYM) &&
              book_alloc(b, &cb.lut, R * CO3_LUT_SIZE) && book_alloc(b, &cb.lut_long, R * (size_t)cb.long_stride) &&
              book_alloc(b, &cb.first, R * (CO3_MAXLEN + 1)) && book_alloc(b, &cb.count, R * (CO3_MAXLEN + 1)) &&
              book_alloc(b, &cb.offs, R * (CO3_MAXLEN + 1)) && book_alloc(b, &cb.perm, R * CO3_MAXSYM) &&
              book_alloc(b, &cb.ksign, (size_t)CO3_MAXSYM);
    if (!ok) { book_free(b); return CO3_ENOMEM; }
    pl->dev.cb = cb;
    if (co3_build_codebook(pl, 0) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        (void)cudaGetLastError();
        book_free(b);
        return CO3_ECUDA;
    }
    cudaFree(cb.cand_len); cudaFree(cb.cand_max);        // build scratch (the first two allocations)
    b.allocs[0] = b.allocs[1] = nullptr;
    b.cb.cand_len = nullptr; b.cb.cand_max = nullptr;
    pl->dev.cb = b.cb;
    b.device = pl->device; b.E = E; b.M = M; b.refs = 1;
    pl->book = &b;
    return CO3_OK;
}

void book_release(co3_plan* pl) {
    if (!pl->book) return;
    std::lock_guard<std::mutex> lock(g_books_mutex);
    SharedBook& b = *static_cast<SharedBook*>(pl->book);
    if (--b.refs == 0) book_free(b);
    pl->book = nullptr;
}

// cudaFuncSetAttribute applies to the current device: one flag per device, set under a lock
constexpr int MAX_DEVICES = 64;
bool g_kernels_ready[MAX_DEVICES];
std::mutex g_kernels_mutex;

cudaError_t setup_kernels_once(int device) {
    std::lock_guard<std::mutex> lock(g_kernels_mutex);
    if (device >= 0 && device < MAX_DEVICES && g_kernels_ready[device]) return cudaSuccess;
    cudaError_t e = co3_setup_kernels();
    if (e == cudaSuccess) e = co3_setup_decode_kernels();
    if (e == cudaSuccess && device >= 0 && device < MAX_DEVICES) g_kernels_ready[device] = true;
    return e;
}

cudaError_t create_host_pipe(co3_plan* pl) {      // co3_iteration_host: copy streams and ordering events
    cudaError_t e = cudaStreamCreateWithFlags(&pl->s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&pl->s_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&pl->ev_h2d, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&pl->ev_conv, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&pl->ev_dec, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&pl->ev_d2h, cudaEventDisableTiming);
    return e;
}

}  // namespace

#define CO3_SYNC_OR_FAIL(pl) do { if (cudaStreamSynchronize((pl)->last_stream) != cudaSuccess) { (void)cudaGetLastError(); return CO3_ECUDA; } } while (0)

extern "C" const char* co3_strerror(int code) {
    switch (code) {
        case CO3_OK: return "ok";
        case CO3_EINVAL: return "invalid argument or unsupported configuration";
        case CO3_ENOMEM: return "out of memory";
        case CO3_ECUDA: return "CUDA runtime error";
        case CO3_ECAPACITY: return "payload exceeds cap_words";
        case CO3_ECORRUPT: return "stream does not decode to its recorded lengths";
        case CO3_ENONFINITE: return "non-finite value in g + gamma*m";
        case CO3_ELIMIT: return "input exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown error";
    }
}

static void free_events(co3_plan* pl) {
    if (pl->prof_ev) {
        for (size_t i = 0; i < (size_t)CO3_NUM_KERNELS * pl->prof_cap * 2; ++i) cudaEventDestroy(pl->prof_ev[i]);
        free(pl->prof_ev);
    }
    pl->prof_ev = nullptr; pl->prof_cap = 0; pl->prof_mask = 0;
    memset(pl->prof_n, 0, sizeof(pl->prof_n));
}

extern "C" int co3_profile_enable(co3_plan* pl, uint32_t kernel_mask, int32_t max_records) {
    if (!pl || max_records < 0 || max_records > (1 << 20)) return CO3_EINVAL;
    CO3_SYNC_OR_FAIL(pl);
    free_events(pl);
    if (!kernel_mask || !max_records) return CO3_OK;
    const size_t n = (size_t)CO3_NUM_KERNELS * max_records * 2;
    pl->prof_ev = (cudaEvent_t*)calloc(n, sizeof(cudaEvent_t));
    if (!pl->prof_ev) return CO3_ENOMEM;
    pl->prof_cap = max_records;
    for (size_t i = 0; i < n; ++i)
        if (cudaEventCreate(&pl->prof_ev[i]) != cudaSuccess) { (void)cudaGetLastError(); free_events(pl); return CO3_ECUDA; }
    pl->prof_mask = kernel_mask;
    return CO3_OK;
}

extern "C" int co3_profile_stride(co3_plan* pl, int32_t every) {
    if (!pl || every < 1) return CO3_EINVAL;
    pl->prof_every = every;
    for (int k = 0; k < CO3_NUM_KERNELS; ++k) pl->prof_seen[k] = 0;
    return CO3_OK;
}

extern "C" int co3_profile_collect(co3_plan* pl, double* total_ms, int64_t* launches) {
    if (!pl || !total_ms || !launches) return CO3_EINVAL;
    CO3_SYNC_OR_FAIL(pl);
    for (int k = 0; k < CO3_NUM_KERNELS; ++k) {
        double tot = 0.0;
        for (int i = 0; i < pl->prof_n[k]; ++i) {
            float ms = 0.0f;
            const size_t o = ((size_t)k * pl->prof_cap + i) * 2;
            if (cudaEventElapsedTime(&ms, pl->prof_ev[o], pl->prof_ev[o + 1]) != cudaSuccess) { (void)cudaGetLastError(); return CO3_ECUDA; }
            tot += ms;
        }
        total_ms[k] = tot;
        launches[k] = pl->prof_n[k];
        pl->prof_n[k] = 0;
    }
    return CO3_OK;
}

extern "C" int64_t co3_launch_count(const co3_plan* pl) { return pl ? pl->launches : 0; }

extern "C" void co3_plan_destroy(co3_plan* pl) {
    if (!pl) return;
    free_events(pl);
    if (pl->s_in) cudaStreamDestroy(pl->s_in);
    if (pl->s_out) cudaStreamDestroy(pl->s_out);
    if (pl->ev_h2d) cudaEventDestroy(pl->ev_h2d);
    if (pl->ev_conv) cudaEventDestroy(pl->ev_conv);
    if (pl->ev_dec) cudaEventDestroy(pl->ev_dec);
    if (pl->ev_d2h) cudaEventDestroy(pl->ev_d2h);
    book_release(pl);
    for (int i = 0; i < pl->n_allocs; ++i) cudaFree(pl->allocs[i]);
    free(pl->h_seg_off);
    delete pl;
}

extern "C" int co3_plan_create(co3_plan** out, const co3_config* cfg) {
    if (!out || !cfg) return CO3_EINVAL;
    *out = nullptr;
    const int E = cfg->fmt.exp_bits, M = cfg->fmt.mant_bits;
    if (!co3_host_fmt_ok(cfg->fmt)) return CO3_EINVAL;
    if (cfg->d < 1 || cfg->ld < cfg->d || (cfg->ld & 3) || cfg->n_users < 1) return CO3_EINVAL;
    if (cfg->cap_words < 4 || (cfg->cap_words & 3) || cfg->cap_words > 0xFFFFFFFFLL) return CO3_EINVAL;
    if (cfg->bias_mode != CO3_BIAS_CURRENT && cfg->bias_mode != CO3_BIAS_LAGGED && cfg->bias_mode != CO3_CODE_LAGGED && cfg->bias_mode != CO3_CODE_EMPIRICAL) return CO3_EINVAL;
    if (!(cfg->gamma >= 0.0f) || !(cfg->gamma <= 1.0f)) return CO3_EINVAL;
    if (cfg->bias_rule != CO3_RULE_POLY && cfg->bias_rule != CO3_RULE_OPT) return CO3_EINVAL;
    if (cfg->d > ((int64_t)1 << 31)) return CO3_EINVAL;
    if (((cfg->d + 4095) / 4096 + (cfg->seg_offsets ? cfg->n_segments : 1)) * (int64_t)cfg->n_users > 0x7FFFFFFFLL) return CO3_EINVAL;
    const int nm = E + M, J = 1 << nm, nsym = 2 * J;
    const int64_t Kmax = co3_host_K(M, J - 1);
    if ((int64_t)cfg->n_users * Kmax >= ((int64_t)1 << 24)) return CO3_EINVAL;   // exact integer sums
    const int S = cfg->seg_offsets ? cfg->n_segments : 1;
    if (S < 1 || S > (1 << 20)) return CO3_EINVAL;

    co3_plan* pl = new (std::nothrow) co3_plan();
    if (!pl) return CO3_ENOMEM;
    memset(pl, 0, sizeof(*pl));
    pl->cfg = *cfg;
    { const char* e = getenv("CO3_TWO_PASS"); pl->two_pass_current = e && e[0] == '1'; }
    pl->h_seg_off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(S + 1));
    if (!pl->h_seg_off) { delete pl; return CO3_ENOMEM; }
    if (cfg->seg_offsets) memcpy(pl->h_seg_off, cfg->seg_offsets, sizeof(int64_t) * (size_t)(S + 1));
    else { pl->h_seg_off[0] = 0; pl->h_seg_off[1] = cfg->d; }
    pl->cfg.seg_offsets = pl->h_seg_off;
    pl->cfg.n_segments = S;

    int64_t n_sub = 0;
    const int64_t nc = co3_partition(cfg->d, S, pl->h_seg_off, nullptr, nullptr, nullptr, nullptr, &n_sub);
    if (nc < 1) { co3_plan_destroy(pl); return CO3_EINVAL; }

    int rc = CO3_OK;
    Co3Chunk* h_chunks = (Co3Chunk*)calloc((size_t)nc, sizeof(Co3Chunk));
    int32_t* h_seg = (int32_t*)malloc(sizeof(int32_t) * (size_t)nc);
    int64_t* h_start = (int64_t*)malloc(sizeof(int64_t) * (size_t)nc);
    int64_t* h_end = (int64_t*)malloc(sizeof(int64_t) * (size_t)nc);
    int64_t* h_sub = (int64_t*)malloc(sizeof(int64_t) * (size_t)nc);
    int32_t* h_seg_chunk0 = (int32_t*)malloc(sizeof(int32_t) * (size_t)(S + 1));
    Co3Group* h_groups = (Co3Group*)calloc((size_t)nc, sizeof(Co3Group));
    const uint32_t* wtab = co3_host_weight_table(E, M);
    const double* logr = co3_host_logr_table();
    if (!h_chunks || !h_seg || !h_start || !h_end || !h_sub || !h_seg_chunk0 || !h_groups || !wtab || !logr) rc = CO3_ENOMEM;

    int64_t n_groups = 0, worst = 0;
    if (rc == CO3_OK) {
        co3_partition(cfg->d, S, pl->h_seg_off, h_seg, h_start, h_end, h_sub, &n_sub);
        int seg_cursor = 0;
        for (int64_t c = 0; c < nc; ++c) {
            h_chunks[c].start = h_start[c];
            h_chunks[c].len = (int32_t)(h_end[c] - h_start[c]);
            h_chunks[c].seg = h_seg[c];
            h_chunks[c].sub0 = (int32_t)h_sub[c];
            worst += 4 * ((16 * (int64_t)h_chunks[c].len + 127) / 128);
            while (seg_cursor <= h_seg[c]) h_seg_chunk0[seg_cursor++] = (int32_t)c;
        }
        while (seg_cursor <= S) h_seg_chunk0[seg_cursor++] = (int32_t)nc;
        const int cpg = cfg->n_users <= 8 ? 8 / cfg->n_users : 1;
        for (int64_t c = 0; c < nc;) {
            int cnt = 1;
            while (cnt < cpg && c + cnt < nc && h_seg[c + cnt] == h_seg[c]) ++cnt;
            h_groups[n_groups].chunk0 = (int32_t)c;
            h_groups[n_groups].count = cnt;
            h_groups[n_groups].seg = h_seg[c];
            ++n_groups;
            c += cnt;
        }
    }

    Co3Dev& dv = pl->dev;
    if (rc == CO3_OK) {
        cudaGetDevice(&pl->device);
        cudaDeviceGetAttribute(&pl->num_sms, cudaDevAttrMultiProcessorCount, pl->device);
        if (pl->num_sms < 1) rc = CO3_ECUDA;
    }
    if (rc == CO3_OK) {
        dv.E = E; dv.M = M; dv.nm = nm; dv.nsym = nsym; dv.J = J; dv.cF = co3_host_cF(E, M);
        dv.Kmax = (uint32_t)Kmax;
        dv.b_lo = -120 - dv.cF;
        int bl = 0;
        while ((Kmax >> bl) != 0) ++bl;
        dv.b_hi = (100 - bl) - dv.cF;
        dv.U = cfg->n_users; dv.S = S; dv.d = cfg->d; dv.ld = cfg->ld;
        dv.u_base = 0; dv.u_count = cfg->n_users;
        dv.sld = (cfg->d + CO3_TILE - 1) / CO3_TILE * CO3_TILE;
        dv.n_chunks = nc; dv.n_sub = n_sub; dv.n_groups = n_groups; dv.cap_words = cfg->cap_words;
        dv.gamma = cfg->gamma;
        pl->worst_case_words = worst;

        Co3Chunk* d_chunks = nullptr; Co3Group* d_groups = nullptr; int64_t* d_seg_off = nullptr;
        int32_t* d_seg_chunk0 = nullptr; uint32_t* d_wtab = nullptr; double* d_logr = nullptr;
        const size_t items = (size_t)nc * (size_t)dv.U;
        int a = 0;
        a |= dev_alloc(pl, &d_chunks, (size_t)nc);
        a |= dev_alloc(pl, &d_groups, (size_t)n_groups);
        a |= dev_alloc(pl, &d_seg_off, (size_t)S + 1);
        a |= dev_alloc(pl, &d_seg_chunk0, (size_t)S + 1);
        a |= dev_alloc(pl, &d_wtab, (size_t)CO3_NIBETA * CO3_NIR * J);
        a |= dev_alloc(pl, &d_logr, 2 * ((size_t)CO3_FIT_GRID + 1));
        const bool code_lagged = cfg->bias_mode == CO3_CODE_LAGGED;   // no stored symbols, staging slots instead
        if (!code_lagged) a |= dev_alloc(pl, &dv.sym, (size_t)dv.U * (size_t)dv.sld);
        else a |= dev_alloc(pl, &dv.slot_buf, items * (size_t)CO3_SLOT_WORDS);
        a |= dev_alloc(pl, &dv.hdr_cur, (size_t)S);
        // Blocks add their shared-memory histograms to global memory with atomics; one counter takes
        // ~1e8 atomics/s, which a large layer converted at full HBM rate exceeds, so the blocks are
        // spread over several copies of the histogram (summed at read-out).
        dv.hist_copies = S <= 1024 ? 8 : 1;
        a |= dev_alloc(pl, &dv.hist, (size_t)dv.hist_copies * S * CO3_MAXSYM + 1);
        a |= dev_alloc(pl, &dv.part_s1, items);
        a |= dev_alloc(pl, &dv.part_s2, items);
        a |= dev_alloc(pl, &dv.part_nf, items);
        a |= dev_alloc(pl, &dv.fit, (size_t)S * 5);
        {   // segments with more than 2^15 (user, chunk) pairs: sum their partials in slices first
            int64_t max_pairs = 0;
            for (int l = 0; l < S; ++l) {
                const int64_t pairs = (int64_t)(h_seg_chunk0[l + 1] - h_seg_chunk0[l]) * dv.U;
                if (pairs > max_pairs) max_pairs = pairs;
            }
            dv.red_k = 0;
            if (max_pairs > (1 << 15)) {
                const int64_t k = (max_pairs + 8191) / 8192;
                dv.red_k = (int)(k > 512 ? 512 : k);
                a |= dev_alloc(pl, &dv.red_s1, (size_t)S * dv.red_k);
                a |= dev_alloc(pl, &dv.red_s2, (size_t)S * dv.red_k);
                a |= dev_alloc(pl, &dv.red_nf, (size_t)S * dv.red_k);
            }
        }
        a |= dev_alloc(pl, &dv.bias_cur, (size_t)S);
        a |= dev_alloc(pl, &dv.spec, 4);
        a |= dev_alloc(pl, &dv.redo_seg, (size_t)S);
        a |= dev_alloc(pl, &dv.redo_old, (size_t)S);
        a |= dev_alloc(pl, &dv.side, (size_t)CO3_SIDE_CAP);
        a |= dev_alloc(pl, &pl->ext_mom, (size_t)S * 3);
        a |= dev_alloc(pl, &pl->fit_ovr, (size_t)S * 2);
        dv.spin_limit = 1 << 20;
        int16_t* d_opt = nullptr;
        const int16_t* h_opt = co3_host_bias_opt_table(E, M);
        a |= dev_alloc(pl, &d_opt, (size_t)CO3_NIBETA * 8);
        if (!h_opt) a = 1;
        dv.bias_rule = cfg->bias_rule;
        a |= dev_alloc(pl, &dv.chunk_words, items);
        a |= dev_alloc(pl, &dv.chunk_bits, items);
        a |= dev_alloc(pl, &dv.user_ovf, (size_t)dv.U);
        {   // one allocation: group totals (u64), published chunk counts (u32), ticket (u32)
            dv.n_grp = (nc + 63) / 64;
            const size_t grp_n = (size_t)dv.U * (size_t)dv.n_grp;
            pl->enc_sync_bytes = (sizeof(unsigned long long) * grp_n + sizeof(uint32_t) * (items + 2) + 7) / 8 * 8;
            dv.enc_sync_words64 = pl->enc_sync_bytes / 8;
            unsigned char* raw = nullptr;
            a |= dev_alloc(pl, &raw, pl->enc_sync_bytes);
            dv.enc_grp = reinterpret_cast<unsigned long long*>(raw);
            dv.enc_st = reinterpret_cast<uint32_t*>(raw + sizeof(unsigned long long) * grp_n);
            dv.enc_ticket = dv.enc_st + items;
        }
        a |= dev_alloc(pl, &dv.flags, 1);
        a |= dev_alloc(pl, &dv.nonfinite_total, 1);
        if (cfg->bias_mode == CO3_CODE_EMPIRICAL) a |= alloc_codebook(pl, pl->cb_emp, (size_t)S, CO3_NCAND_HIST);
        if (a) rc = CO3_ENOMEM;
        if (rc == CO3_OK) {
            cudaError_t e = cudaSuccess;
            auto up = [&](void* dst, const void* src, size_t bytes) {
                if (e == cudaSuccess) e = cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice);
            };
            up(d_chunks, h_chunks, sizeof(Co3Chunk) * (size_t)nc);
            up(d_groups, h_groups, sizeof(Co3Group) * (size_t)n_groups);
            up(d_seg_off, pl->h_seg_off, sizeof(int64_t) * (size_t)(S + 1));
            up(d_seg_chunk0, h_seg_chunk0, sizeof(int32_t) * (size_t)(S + 1));
            up(d_wtab, wtab, sizeof(uint32_t) * (size_t)CO3_NIBETA * CO3_NIR * J);
            up(d_logr, logr, sizeof(double) * 2 * ((size_t)CO3_FIT_GRID + 1));
            up(d_opt, h_opt, sizeof(int16_t) * (size_t)CO3_NIBETA * 8);
            dv.bias_opt_tab = d_opt;
            if (e == cudaSuccess) e = cudaMemset(dv.flags, 0, sizeof(uint32_t));
            if (e == cudaSuccess) e = cudaMemset(dv.nonfinite_total, 0, sizeof(unsigned long long));
            if (e == cudaSuccess) e = cudaMemset(dv.bias_cur, 0, sizeof(int32_t) * (size_t)S);
            if (e == cudaSuccess) e = cudaMemset(dv.spec, 0, sizeof(int32_t) * 4);
            if (e == cudaSuccess) e = cudaMemset(dv.fit, 0, sizeof(double) * (size_t)S * 5);
            if (e == cudaSuccess) e = cudaMemset(dv.hist, 0, sizeof(unsigned long long) * ((size_t)dv.hist_copies * S * CO3_MAXSYM + 1));
            dv.ticket = reinterpret_cast<unsigned int*>(dv.hist + (size_t)dv.hist_copies * S * CO3_MAXSYM);
            if (e == cudaSuccess && dv.sym) e = cudaMemset(dv.sym, 0, (size_t)dv.U * (size_t)dv.sld);
            if (e == cudaSuccess) e = cudaMemset(dv.hdr_cur, 0, sizeof(co3_seg_header) * (size_t)S);
            if (e == cudaSuccess) e = setup_kernels_once(pl->device);
            if (e == cudaSuccess) e = create_host_pipe(pl);
            pl->host_pipe_ready = (e == cudaSuccess);
            if (e != cudaSuccess) { (void)cudaGetLastError(); rc = CO3_ECUDA; }
            if (e == cudaSuccess) {                  // the decoder's work split (needs the kernels' attributes set)
                const int max_blocks = co3_decode_max_blocks(dv.U, pl->num_sms);
                int32_t* h_part = (int32_t*)malloc(sizeof(int32_t) * (size_t)(max_blocks + 1));
                int32_t* d_part = nullptr;
                if (!h_part || dev_alloc(pl, &d_part, (size_t)max_blocks + 1) != CO3_OK) rc = CO3_ENOMEM;
                else {
                    dv.dec_blocks = co3_decode_partition(h_chunks, nc, h_groups, n_groups, dv.U, max_blocks, h_part);
                    e = cudaMemcpy(d_part, h_part, sizeof(int32_t) * (size_t)(max_blocks + 1), cudaMemcpyHostToDevice);
                    dv.dec_part = d_part;
                    if (dv.dec_blocks < 1) rc = CO3_ENOMEM;
                    if (e != cudaSuccess) { (void)cudaGetLastError(); rc = CO3_ECUDA; }
                }
                free(h_part);
            }
            dv.chunks = d_chunks; dv.groups = d_groups; dv.seg_off = d_seg_off;
            dv.seg_chunk0 = d_seg_chunk0; dv.wtab = d_wtab; dv.logr_tab = d_logr;
            if (rc == CO3_OK) rc = book_acquire(pl);  // Huffman codes of all model rows: built once per device and format
        }
    }
    free(h_chunks); free(h_seg); free(h_start); free(h_end); free(h_sub); free(h_seg_chunk0); free(h_groups);
    if (rc != CO3_OK) { co3_plan_destroy(pl); return rc; }
    *out = pl;
    return CO3_OK;
}

extern "C" int co3_sizes(const co3_plan* pl, int64_t* n_chunks, int64_t* n_sub, int64_t* worst_case_words) {
    if (!pl) return CO3_EINVAL;
    if (n_chunks) *n_chunks = pl->dev.n_chunks;
    if (n_sub) *n_sub = pl->dev.n_sub;
    if (worst_case_words) *worst_case_words = pl->worst_case_words;
    return CO3_OK;
}

#define CO3_TRY(call) do { if ((call) != cudaSuccess) { (void)cudaGetLastError(); return CO3_ECUDA; } } while (0)

extern "C" int co3_encode(co3_plan* pl, const float* grad, float* residual, uint32_t* bitstream,
                          uint16_t* sub_bits, uint32_t* chunk_off, uint64_t* user_bits,
                          co3_seg_header* hdr, void* cuda_stream) {
    if (!pl || !grad || !residual || !bitstream || !sub_bits || !chunk_off || !user_bits || !hdr) return CO3_EINVAL;
    if (((uintptr_t)grad | (uintptr_t)residual | (uintptr_t)bitstream) & 15) return CO3_EINVAL;
    if (pl->cfg.bias_mode == CO3_CODE_EMPIRICAL && !pl->emp_lens) return CO3_EINVAL;   // use co3_encode_empirical
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    if (pl->cfg.bias_mode == CO3_CODE_LAGGED) {
        // The header of this iteration was fixed by the previous one (at t = 0: by a statistics pass),
        // so conversion and packing are one pass; the fit that follows prepares the next iteration.
        if (pl->iteration == 0) {
            CO3_TRY(co3_launch_stats(pl, grad, residual, 0, pl->dev.U, st));
            CO3_TRY(co3_launch_fit(pl, 2, pl->dev.hdr_cur, st));
        }
        CO3_TRY(cudaMemcpyAsync(hdr, pl->dev.hdr_cur, sizeof(co3_seg_header) * (size_t)pl->dev.S, cudaMemcpyDeviceToDevice, st));
        CO3_TRY(co3_launch_convert_pack(pl, grad, residual, sub_bits, st));
        if (pl->record_conv) CO3_TRY(cudaEventRecord(pl->ev_conv, st));
        CO3_TRY(co3_launch_scan_gather(pl, bitstream, sub_bits, chunk_off, (unsigned long long*)user_bits, st));
        CO3_TRY(co3_launch_fit(pl, 3, pl->dev.hdr_cur, st));
        pl->iteration++;
        return CO3_OK;
    }
    // Bias from the current moments: the fit after the statistics pass also gives the header (the convert
    // pass would hand the next fit the same sums), so there is one fit per iteration in both modes.
    const bool current = pl->cfg.bias_mode == CO3_BIAS_CURRENT;
    if (current && pl->iteration > 0 && !pl->two_pass_current) {
        // The bias of this iteration comes from this iteration's own moments, and those ride along with
        // the convert pass: convert under the previous iteration's bias, fit, and convert again only
        // the layers whose bias came out different (co3_launch_reconvert) -- the results are those of
        // the statistics-pass-first order, bit for bit, at the cost of the lagged bias.
        CO3_TRY(co3_launch_convert(pl, grad, residual, 0, pl->dev.U, true, st, false, true));
        if (pl->record_conv) CO3_TRY(cudaEventRecord(pl->ev_conv, st));
        CO3_TRY(co3_launch_fit(pl, 6, hdr, st, false, residual));
        CO3_TRY(co3_launch_reconvert(pl, residual, st));
        CO3_TRY(co3_launch_encode(pl, hdr, bitstream, sub_bits, chunk_off, (unsigned long long*)user_bits, st));
        pl->iteration++;
        return CO3_OK;
    }
    const bool with_stats = pl->iteration == 0 || current;
    if (with_stats) {
        CO3_TRY(co3_launch_stats(pl, grad, residual, 0, pl->dev.U, st));
        CO3_TRY(co3_launch_fit(pl, current ? 5 : 0, hdr, st, true));   // also zeroes the convert pass's histogram and ticket
    }
    CO3_TRY(co3_launch_convert(pl, grad, residual, 0, pl->dev.U, true, st, with_stats));
    if (pl->record_conv) CO3_TRY(cudaEventRecord(pl->ev_conv, st));   // the gradient buffer is free from here on
    if (!current) CO3_TRY(co3_launch_fit(pl, 1, hdr, st));
    if (pl->cfg.bias_mode == CO3_CODE_EMPIRICAL) CO3_TRY(co3_build_hist_codes(pl, pl->emp_lens, st));
    CO3_TRY(co3_launch_encode(pl, hdr, bitstream, sub_bits, chunk_off, (unsigned long long*)user_bits, st));
    pl->iteration++;
    return CO3_OK;
}

// ---- one iteration in tiles of users (gradients that do not fit the device at once) -------------
// A statistics pass in front of the conversion: at t = 0, and in every iteration of the current-moments bias
// in its two-pass form; else that bias converts under the previous one and repairs (see co3_encode).
static bool tiled_needs_statistics(const co3_plan* pl) {
    return pl->iteration == 0 || (pl->cfg.bias_mode == CO3_BIAS_CURRENT && pl->two_pass_current);
}

extern "C" int co3_tiled_begin(co3_plan* pl, int32_t* need_statistics) {
    if (!pl || !need_statistics) return CO3_EINVAL;
    if (pl->cfg.bias_mode != CO3_BIAS_CURRENT && pl->cfg.bias_mode != CO3_BIAS_LAGGED) return CO3_EINVAL;
    pl->tiled_state = 1;
    pl->tiled_users = 0;
    pl->use_ext_mom = false;
    *need_statistics = tiled_needs_statistics(pl) ? 1 : 0;
    return CO3_OK;
}

static int tile_args_ok(const co3_plan* pl, const float* grad_tile, const float* residual, int32_t user0, int32_t n) {
    if (!pl || !grad_tile || !residual || user0 < 0 || n < 1 || user0 + n > pl->dev.U) return 0;
    if (((uintptr_t)grad_tile | (uintptr_t)residual) & 15) return 0;
    return 1;
}

extern "C" int co3_tiled_statistics(co3_plan* pl, const float* grad_tile, const float* residual, int32_t user0,
                                    int32_t n_tile_users, void* cuda_stream) {
    if (!tile_args_ok(pl, grad_tile, residual, user0, n_tile_users)) return CO3_EINVAL;
    if (pl->tiled_state != 1 && pl->tiled_state != 2) return CO3_EINVAL;       // before any convert tile
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    CO3_TRY(co3_launch_stats(pl, grad_tile, residual, user0, n_tile_users, st));
    pl->tiled_state = 2;
    return CO3_OK;
}

extern "C" int co3_tiled_convert(co3_plan* pl, const float* grad_tile, float* residual, int32_t user0,
                                 int32_t n_tile_users, void* cuda_stream) {
    if (!tile_args_ok(pl, grad_tile, residual, user0, n_tile_users)) return CO3_EINVAL;
    if (pl->tiled_state < 1) return CO3_EINVAL;
    const bool need_stats = tiled_needs_statistics(pl);
    const bool guess = pl->cfg.bias_mode == CO3_BIAS_CURRENT && !need_stats;
    if (pl->tiled_state == 1 && need_stats) return CO3_EINVAL;                 // the statistics tiles come first
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    const bool first = pl->tiled_state != 3;
    if (first && need_stats) CO3_TRY(co3_launch_fit(pl, 0, nullptr, st));       // bias from the pooled statistics
    CO3_TRY(co3_launch_convert(pl, grad_tile, residual, user0, n_tile_users, first, st, false, guess));
    pl->tiled_residual = residual;
    pl->tiled_state = 3;
    pl->tiled_users += n_tile_users;
    return CO3_OK;
}

extern "C" int co3_tiled_finish(co3_plan* pl, uint32_t* bitstream, uint16_t* sub_bits, uint32_t* chunk_off,
                                uint64_t* user_bits, co3_seg_header* hdr, void* cuda_stream) {
    if (!pl || !bitstream || !sub_bits || !chunk_off || !user_bits || !hdr) return CO3_EINVAL;
    if ((uintptr_t)bitstream & 15) return CO3_EINVAL;
    if (pl->tiled_state != 3 || pl->tiled_users != pl->dev.U) return CO3_EINVAL;   // every user exactly once
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    if (pl->cfg.bias_mode == CO3_BIAS_CURRENT && !tiled_needs_statistics(pl)) {
        CO3_TRY(co3_launch_fit(pl, 6, hdr, st, false, pl->tiled_residual));     // the tiles were converted under the previous bias
        CO3_TRY(co3_launch_reconvert(pl, pl->tiled_residual, st));
    } else {
        CO3_TRY(co3_launch_fit(pl, 1, hdr, st));
    }
    CO3_TRY(co3_launch_encode(pl, hdr, bitstream, sub_bits, chunk_off, (unsigned long long*)user_bits, st));
    pl->iteration++;
    pl->tiled_state = 0;
    return CO3_OK;
}

// ---- pooled moments across plans (slices of d) ---------------------------------------------------
extern "C" int co3_moments_export(co3_plan* pl, double* moments, void* cuda_stream) {
    if (!pl || !moments) return CO3_EINVAL;
    if (pl->tiled_state != 2 && pl->tiled_state != 3) return CO3_EINVAL;
    if (pl->tiled_state == 3 && pl->tiled_users != pl->dev.U) return CO3_EINVAL;   // every user converted
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    pl->mom_out = moments;
    CO3_TRY(co3_launch_fit(pl, 4, nullptr, st));
    pl->mom_out = nullptr;
    return CO3_OK;
}

extern "C" int co3_moments_import(co3_plan* pl, const double* moments, void* cuda_stream) {
    if (!pl || !moments) return CO3_EINVAL;
    if (pl->tiled_state != 2 && pl->tiled_state != 3) return CO3_EINVAL;
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    CO3_TRY(cudaMemcpyAsync(pl->ext_mom, moments, sizeof(double) * 3 * (size_t)pl->dev.S, cudaMemcpyDeviceToDevice, st));
    pl->use_ext_mom = true;
    return CO3_OK;
}

extern "C" int co3_encode_empirical(co3_plan* pl, const float* grad, float* residual, uint32_t* bitstream,
                                    uint16_t* sub_bits, uint32_t* chunk_off, uint64_t* user_bits,
                                    co3_seg_header* hdr, uint8_t* code_lens, void* cuda_stream) {
    if (!pl || !code_lens || pl->cfg.bias_mode != CO3_CODE_EMPIRICAL) return CO3_EINVAL;
    pl->emp_lens = code_lens;
    const int rc = co3_encode(pl, grad, residual, bitstream, sub_bits, chunk_off, user_bits, hdr, cuda_stream);
    pl->emp_lens = nullptr;
    return rc;
}

extern "C" int co3_decode_aggregate(co3_plan* pl, const uint32_t* bitstream, const uint16_t* sub_bits,
                                    const uint32_t* chunk_off, const co3_seg_header* hdr, float* avg_grad,
                                    void* cuda_stream) {
    if (!pl || !bitstream || !sub_bits || !chunk_off || !hdr || !avg_grad) return CO3_EINVAL;
    if ((uintptr_t)bitstream & 15) return CO3_EINVAL;
    if (pl->cfg.bias_mode == CO3_CODE_EMPIRICAL && !pl->emp_lens_in) return CO3_EINVAL;   // use ..._empirical
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    if (pl->cfg.bias_mode == CO3_CODE_EMPIRICAL) CO3_TRY(co3_build_codes_from_lens(pl, pl->emp_lens_in, st));
    CO3_TRY(co3_launch_decode(pl, bitstream, sub_bits, chunk_off, hdr, avg_grad, nullptr, 0.0f, st));
    return CO3_OK;
}

extern "C" int co3_decode_aggregate_empirical(co3_plan* pl, const uint32_t* bitstream, const uint16_t* sub_bits,
                                              const uint32_t* chunk_off, const co3_seg_header* hdr,
                                              const uint8_t* code_lens, float* avg_grad, void* cuda_stream) {
    if (!pl || !code_lens || pl->cfg.bias_mode != CO3_CODE_EMPIRICAL) return CO3_EINVAL;
    pl->emp_lens_in = code_lens;
    const int rc = co3_decode_aggregate(pl, bitstream, sub_bits, chunk_off, hdr, avg_grad, cuda_stream);
    pl->emp_lens_in = nullptr;
    return rc;
}

extern "C" int co3_decode_aggregate_update(co3_plan* pl, const uint32_t* bitstream, const uint16_t* sub_bits,
                                           const uint32_t* chunk_off, const co3_seg_header* hdr, float* avg_grad,
                                           float* weights, float step, void* cuda_stream) {
    if (!pl || !bitstream || !sub_bits || !chunk_off || !hdr || !avg_grad || !weights) return CO3_EINVAL;
    if ((uintptr_t)bitstream & 15 || pl->cfg.bias_mode == CO3_CODE_EMPIRICAL) return CO3_EINVAL;
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    CO3_TRY(co3_launch_decode(pl, bitstream, sub_bits, chunk_off, hdr, avg_grad, weights, step, st));
    return CO3_OK;
}

extern "C" int co3_iteration_host(co3_plan* pl, const float* h_grad, float* d_grad, float* d_residual,
                                  uint32_t* d_bitstream, uint16_t* d_sub_bits, uint32_t* d_chunk_off,
                                  uint64_t* d_user_bits, co3_seg_header* d_hdr, float* d_avg, float* h_avg,
                                  void* cuda_stream) {
    if (!pl || !h_grad || !d_grad || !h_avg || !d_avg) return CO3_EINVAL;
    cudaStream_t st = as_stream(cuda_stream);
    // The copies run on two streams of the plan so that consecutive calls overlap: the gradient of
    // call k+1 goes to the device while call k is still encoding, decoding and copying its average
    // back (PCIe is full duplex).  d_grad is free as soon as the convert pass of the previous call
    // has read it; everything else is ordered through the caller's stream, which at the end of the
    // call also waits for the copy of the average, so synchronising it is still all the caller does.
    if (!pl->host_pipe_ready) return CO3_ECUDA;       // (its streams and events are made by co3_plan_create)
    if (pl->ev_conv_recorded) CO3_TRY(cudaStreamWaitEvent(pl->s_in, pl->ev_conv, 0));
    CO3_TRY(cudaMemcpyAsync(d_grad, h_grad, sizeof(float) * (size_t)pl->dev.U * (size_t)pl->dev.ld,
                            cudaMemcpyHostToDevice, pl->s_in));
    CO3_TRY(cudaEventRecord(pl->ev_h2d, pl->s_in));
    CO3_TRY(cudaStreamWaitEvent(st, pl->ev_h2d, 0));
    pl->record_conv = true;
    int rc = co3_encode(pl, d_grad, d_residual, d_bitstream, d_sub_bits, d_chunk_off, d_user_bits, d_hdr, cuda_stream);
    pl->record_conv = false;
    if (rc != CO3_OK) return rc;
    pl->ev_conv_recorded = true;
    rc = co3_decode_aggregate(pl, d_bitstream, d_sub_bits, d_chunk_off, d_hdr, d_avg, cuda_stream);
    if (rc != CO3_OK) return rc;
    CO3_TRY(cudaEventRecord(pl->ev_dec, st));
    CO3_TRY(cudaStreamWaitEvent(pl->s_out, pl->ev_dec, 0));
    CO3_TRY(cudaMemcpyAsync(h_avg, d_avg, sizeof(float) * (size_t)pl->dev.d, cudaMemcpyDeviceToHost, pl->s_out));
    CO3_TRY(cudaEventRecord(pl->ev_d2h, pl->s_out));
    CO3_TRY(cudaStreamWaitEvent(st, pl->ev_d2h, 0));
    return CO3_OK;
}

extern "C" int co3_status(co3_plan* pl, uint32_t* flags, uint64_t* nonfinite_count, int32_t clear) {
    if (!pl) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    uint32_t f = 0;
    unsigned long long n = 0;
    CO3_TRY(cudaMemcpy(&f, pl->dev.flags, sizeof(f), cudaMemcpyDeviceToHost));
    CO3_TRY(cudaMemcpy(&n, pl->dev.nonfinite_total, sizeof(n), cudaMemcpyDeviceToHost));
    if (flags) *flags = f;
    if (nonfinite_count) *nonfinite_count = n;
    if (clear) {
        CO3_TRY(cudaMemset(pl->dev.flags, 0, sizeof(uint32_t)));
        CO3_TRY(cudaMemset(pl->dev.nonfinite_total, 0, sizeof(unsigned long long)));
    }
    return CO3_OK;
}

extern "C" int co3_get_fit(co3_plan* pl, int32_t seg, double* beta, double* alpha, double* N, double* S1,
                           double* S2) {
    if (!pl || seg < 0 || seg >= pl->dev.S) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    double f[5];
    CO3_TRY(cudaMemcpy(f, pl->dev.fit + 5 * (size_t)seg, sizeof(f), cudaMemcpyDeviceToHost));
    if (beta) *beta = f[0];
    if (alpha) *alpha = f[1];
    if (N) *N = f[2];
    if (S1) *S1 = f[3];
    if (S2) *S2 = f[4];
    return CO3_OK;
}

extern "C" int co3_state_export(co3_plan* pl, int64_t* iteration, int32_t* next_bias) {
    if (!pl || !iteration || !next_bias) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    CO3_TRY(cudaMemcpy(next_bias, pl->dev.bias_cur, sizeof(int32_t) * (size_t)pl->dev.S, cudaMemcpyDeviceToHost));
    *iteration = pl->iteration;
    return CO3_OK;
}

extern "C" int co3_state_import(co3_plan* pl, int64_t iteration, const int32_t* next_bias) {
    if (!pl || !next_bias || iteration < 0) return CO3_EINVAL;
    for (int l = 0; l < pl->dev.S; ++l)
        if (next_bias[l] < pl->dev.b_lo || next_bias[l] > pl->dev.b_hi) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    CO3_TRY(cudaMemcpy(pl->dev.bias_cur, next_bias, sizeof(int32_t) * (size_t)pl->dev.S, cudaMemcpyHostToDevice));
    pl->iteration = iteration;
    return CO3_OK;
}

extern "C" int co3_state_header(co3_plan* pl, int32_t import, co3_seg_header* next_header) {
    if (!pl || !next_header) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    const size_t bytes = sizeof(co3_seg_header) * (size_t)pl->dev.S;
    if (import) {
        for (int l = 0; l < pl->dev.S; ++l) {
            bool bad = false;
            (void)co3_row_of(next_header[l], &bad);
            if (bad || next_header[l].bias < pl->dev.b_lo || next_header[l].bias > pl->dev.b_hi) return CO3_EINVAL;
        }
        CO3_TRY(cudaMemcpy(pl->dev.hdr_cur, next_header, bytes, cudaMemcpyHostToDevice));
    } else {
        CO3_TRY(cudaMemcpy(next_header, pl->dev.hdr_cur, bytes, cudaMemcpyDeviceToHost));
    }
    return CO3_OK;
}

extern "C" int co3_set_fit_override(co3_plan* pl, const double* fit) {
    if (!pl) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    pl->use_fit_ovr = false;
    if (!fit) return CO3_OK;
    for (int l = 0; l < pl->dev.S; ++l)
        if (!(fit[2 * l] > 0.0) || !(fit[2 * l + 1] >= 0.0) || !(fit[2 * l + 1] < 1e300)) return CO3_EINVAL;
    CO3_TRY(cudaMemcpy(pl->fit_ovr, fit, sizeof(double) * 2 * (size_t)pl->dev.S, cudaMemcpyHostToDevice));
    pl->use_fit_ovr = true;
    return CO3_OK;
}

extern "C" int co3_debug_encode_stalled(co3_plan* pl, uint32_t* bitstream, uint16_t* sub_bits, uint32_t* chunk_off,
                                        uint64_t* user_bits, const co3_seg_header* hdr, int32_t spin_limit,
                                        void* cuda_stream) {
    if (!pl || !bitstream || !sub_bits || !chunk_off || !user_bits || !hdr) return CO3_EINVAL;
    if ((uintptr_t)bitstream & 15 || spin_limit < 1 || spin_limit > (1 << 20)) return CO3_EINVAL;
    if (!pl->dev.sym || pl->cfg.bias_mode == CO3_CODE_EMPIRICAL || pl->iteration < 1) return CO3_EINVAL;
    if (pl->dev.n_chunks * (int64_t)pl->dev.U < 2) return CO3_EINVAL;
    cudaStream_t st = as_stream(cuda_stream);
    pl->last_stream = st;
    CO3_TRY(co3_launch_encode_stalled(pl, hdr, bitstream, sub_bits, chunk_off, (unsigned long long*)user_bits,
                                      spin_limit, st));
    return CO3_OK;
}

extern "C" int co3_debug_symbols(co3_plan* pl, uint8_t* symbols, void* cuda_stream) {
    if (!pl || !symbols || !pl->dev.sym) return CO3_EINVAL;    // the fully lagged code keeps no symbols
    cudaStream_t st = as_stream(cuda_stream);
    CO3_TRY(co3_launch_symbol_export(pl, symbols, st));
    CO3_TRY(cudaStreamSynchronize(st));
    return CO3_OK;
}

extern "C" int co3_debug_hist(co3_plan* pl, uint64_t* hist) {
    if (!pl || !hist) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    const int S = pl->dev.S, nsym = pl->dev.nsym, nm = pl->dev.nm;
    const int copies = pl->dev.hist_copies;
    const size_t per_copy = (size_t)S * CO3_MAXSYM;
    uint64_t* tmp = (uint64_t*)malloc(sizeof(uint64_t) * per_copy * copies);
    if (!tmp) return CO3_ENOMEM;
    if (cudaMemcpy(tmp, pl->dev.hist, sizeof(uint64_t) * per_copy * copies, cudaMemcpyDeviceToHost) != cudaSuccess) {
        (void)cudaGetLastError();
        free(tmp);
        return CO3_ECUDA;
    }
    for (int l = 0; l < S; ++l)                          // stored by internal symbol, reported by public symbol
        for (int sym = 0; sym < nsym; ++sym)
        {
            uint64_t tot = 0;
            for (int k = 0; k < copies; ++k) tot += tmp[k * per_copy + (size_t)l * CO3_MAXSYM + co3_sym_internal(sym, nm)];
            hist[(size_t)l * nsym + sym] = tot;
        }
    free(tmp);
    return CO3_OK;
}

extern "C" int co3_debug_code(co3_plan* pl, const co3_seg_header* hdr, uint8_t* lengths, uint32_t* codewords) {
    if (!pl || !hdr || !lengths || !codewords) return CO3_EINVAL;
    CO3_TRY(cudaStreamSynchronize(pl->last_stream));
    const int S = pl->dev.S, nsym = pl->dev.nsym;
    co3_seg_header* h = (co3_seg_header*)malloc(sizeof(co3_seg_header) * (size_t)S);
    if (!h) return CO3_ENOMEM;
    int rc = CO3_OK;
    if (cudaMemcpy(h, hdr, sizeof(co3_seg_header) * (size_t)S, cudaMemcpyDeviceToHost) != cudaSuccess) rc = CO3_ECUDA;
    for (int l = 0; l < S && rc == CO3_OK; ++l) {
        bool bad = false;
        const size_t row = (size_t)co3_row_of(h[l], &bad);
        if (bad) { rc = CO3_ECORRUPT; break; }
        if (cudaMemcpy(lengths + (size_t)l * nsym, pl->dev.cb.len_pub + row * CO3_MAXSYM, (size_t)nsym,
                       cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemcpy(codewords + (size_t)l * nsym, pl->dev.cb.code_msb + row * CO3_MAXSYM,
                       sizeof(uint32_t) * (size_t)nsym, cudaMemcpyDeviceToHost) != cudaSuccess)
            rc = CO3_ECUDA;
    }
    free(h);
    if (rc == CO3_ECUDA) (void)cudaGetLastError();
    return rc;
}
