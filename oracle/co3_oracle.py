"""ctypes front end and per-iteration driver of the CO3 CPU oracle (test infrastructure).

The arithmetic lives in co3_oracle.c; this file only sequences the steps of Algorithm 1
(lines 8-10 at the users, lines 13-14 at the parameter server) and keeps the state that the
method carries between iterations (the bias for the next iteration in LAGGED mode).  The one
exception is the model update of line 14 (decode_aggregate_update), two numpy float32 operations
written out here.  The memory m^(u) is the caller's array and is updated in place.
"""
import ctypes as C
import numpy as np

from . import build as _build

_lib = None

MODE_CURRENT = 0   # bias b_t from the moments of a_t itself (a stats pass every iteration)
MODE_LAGGED = 1    # stats pass at t = 0 only; b_t (t >= 1) from the fit of iteration t-1
MODE_EMPIRICAL = 3    # bias as MODE_LAGGED; the code of a layer is the Huffman code of this iteration's symbol
                      # histogram and its length table is side information (no GenNorm model in the code)
MODE_LAGGED_CODE = 2  # as MODE_LAGGED, and the code model of iteration t (t >= 1) is the fit of iteration
                      # t-1 as well: the whole header of iteration t is known before g_t is seen

OK, EINVAL, ECAPACITY, ECORRUPT = 0, -1, -4, -5

_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")
_u64p = np.ctypeslib.ndpointer(np.uint64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(np.int64, flags="C_CONTIGUOUS")
_dp = C.POINTER(C.c_double)
_i64 = C.c_int64


def lib():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(_build.build())
    L.co3o_num_mag.restype = C.c_int
    L.co3o_K.restype = _i64
    L.co3o_K.argtypes = [C.c_int] * 3
    L.co3o_Kmax.restype = _i64
    for n in ("co3o_cF", "co3o_b_lo", "co3o_b_hi"):
        getattr(L, n).restype = C.c_int
        getattr(L, n).argtypes = [C.c_int, C.c_int]
    L.co3o_grid_value.restype = C.c_float
    L.co3o_grid_value.argtypes = [C.c_int] * 4
    L.co3o_quantize_one.restype = C.c_int
    L.co3o_quantize_one.argtypes = [C.c_float, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_float)]
    L.co3o_stats.restype = None
    L.co3o_stats.argtypes = [_f32p, _f32p, C.c_int, _i64, _i64, _i64, C.c_float,
                             _dp, _dp, _dp, C.POINTER(_i64)]
    L.co3o_convert.restype = None
    L.co3o_convert.argtypes = [_f32p, _f32p, _u8p, C.c_int, _i64, _i64, _i64, _i64, C.c_float,
                               C.c_int, C.c_int, C.c_int, _u64p, _dp, _dp, _dp, C.POINTER(_i64)]
    L.co3o_logR.restype = C.c_double
    L.co3o_logR.argtypes = [C.c_double]
    L.co3o_fit.restype = None
    L.co3o_fit.argtypes = [C.c_double] * 3 + [_dp, _dp]
    L.co3o_poly.restype = C.c_double
    L.co3o_poly.argtypes = [C.c_double]
    L.co3o_bias.restype = C.c_int
    L.co3o_bias.argtypes = [C.c_double, C.c_double, C.c_int, C.c_int]
    L.co3o_distortion.restype = C.c_double
    L.co3o_distortion.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
    L.co3o_bias_opt_table.restype = None
    L.co3o_bias_opt_table.argtypes = [C.c_int, C.c_int, C.c_void_p]
    L.co3o_bias_opt.restype = C.c_int
    L.co3o_bias_opt.argtypes = [C.c_double, C.c_double, C.c_int, C.c_int, C.c_void_p]
    L.co3o_header.restype = None
    L.co3o_header.argtypes = [C.c_double, C.c_double, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    L.co3o_gammainc.restype = C.c_double
    L.co3o_gammainc.argtypes = [C.c_double, C.c_double]
    L.co3o_model_weights.restype = C.c_int
    L.co3o_model_weights.argtypes = [C.c_int] * 4 + [_u32p]
    L.co3o_huffman.restype = C.c_int
    L.co3o_huffman.argtypes = [_u32p, C.c_int, _u8p, C.POINTER(C.c_uint32)]
    L.co3o_canonical.restype = None
    L.co3o_canonical.argtypes = [_u8p, C.c_int, _u32p]
    L.co3o_partition.restype = _i64
    L.co3o_partition.argtypes = [_i64, C.c_int, _i64p, C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.POINTER(_i64)]
    L.co3o_encode_user.restype = C.c_int
    L.co3o_encode_user.argtypes = [_u8p, _i64, _i32p, _i64p, _i64p, _i64p, C.c_int, _u8p, _u32p,
                                   _u32p, _i64, _u16p, _u32p, C.POINTER(C.c_uint64)]
    L.co3o_decode_aggregate.restype = C.c_int
    L.co3o_decode_aggregate.argtypes = [_u32p, _i64, _u16p, _i64, _u32p, C.c_int, _i64, _i32p,
                                        _i64p, _i64p, _i64p, C.c_int, _i32p, C.c_int, C.c_int,
                                        _f32p, C.c_void_p, _i64, C.c_void_p]
    L.co3o_huffman_counts.restype = C.c_int
    L.co3o_huffman_counts.argtypes = [np.ctypeslib.ndpointer(np.uint64, flags="C_CONTIGUOUS"), C.c_int, _u8p,
                                      C.POINTER(C.c_uint32)]
    _lib = L
    return L


# ---- thin step wrappers (used by the pins) --------------------------------------------------
def K(E, M, j):
    return int(lib().co3o_K(E, M, j))


def Kmax(E, M):
    return int(lib().co3o_Kmax(E, M))


def cF(E, M):
    return int(lib().co3o_cF(E, M))


def b_range(E, M):
    return int(lib().co3o_b_lo(E, M)), int(lib().co3o_b_hi(E, M))


def grid_value(E, M, b, sym):
    return float(lib().co3o_grid_value(E, M, b, sym))


def quantize_one(a, E, M, b):
    q = C.c_float()
    s = lib().co3o_quantize_one(C.c_float(a), E, M, b, C.byref(q))
    return int(s), float(q.value)


def stats(g, m, lo, hi, gamma):
    U, ld = g.shape
    N, S1, S2, nf = C.c_double(), C.c_double(), C.c_double(), _i64()
    lib().co3o_stats(g, m, U, ld, lo, hi, gamma, C.byref(N), C.byref(S1), C.byref(S2), C.byref(nf))
    return N.value, S1.value, S2.value, nf.value


def convert(g, m, sym, lo, hi, gamma, E, M, b, hist):
    U, ld = g.shape
    N, S1, S2, nf = C.c_double(), C.c_double(), C.c_double(), _i64()
    lib().co3o_convert(g, m, sym, U, ld, sym.shape[1], lo, hi, gamma, E, M, b, hist,
                       C.byref(N), C.byref(S1), C.byref(S2), C.byref(nf))
    return N.value, S1.value, S2.value, nf.value


def logR(beta):
    return lib().co3o_logR(beta)


def fit(N, S1, S2):
    b, a = C.c_double(), C.c_double()
    lib().co3o_fit(N, S1, S2, C.byref(b), C.byref(a))
    return b.value, a.value


def poly(beta):
    return lib().co3o_poly(beta)


def bias(beta, alpha, E, M):
    return int(lib().co3o_bias(beta, alpha, E, M))


RULE_POLY = 0   # the paper's polynomial (Eq. "approximate"), nearest integer exponent
RULE_OPT = 1    # the integer bias that minimises the L2 conversion error of the fitted GenNorm
_OPT_TABLES = {}


def distortion(E, M, ibeta, ir):
    """E[(Q(X) - X)^2] / alpha^2 for X ~ GenNorm(alpha, 2^(ibeta/8)) with log2(alpha) - b = ir/8."""
    return float(lib().co3o_distortion(E, M, ibeta, ir))


def bias_opt_table(E, M):
    """[23][8] int16: best ir for (ibeta + 14, round(8 log2 alpha) mod 8); cached per format."""
    if (E, M) not in _OPT_TABLES:
        tab = np.zeros((23, 8), np.int16)
        lib().co3o_bias_opt_table(E, M, tab.ctypes.data)
        _OPT_TABLES[(E, M)] = tab
    return _OPT_TABLES[(E, M)]


def bias_opt(beta, alpha, E, M):
    tab = bias_opt_table(E, M)
    return int(lib().co3o_bias_opt(beta, alpha, E, M, tab.ctypes.data))


def bias_by_rule(rule, beta, alpha, E, M):
    return bias_opt(beta, alpha, E, M) if rule == RULE_OPT else bias(beta, alpha, E, M)


def header(beta, alpha, b):
    ib, ir = C.c_int(), C.c_int()
    lib().co3o_header(beta, alpha, b, C.byref(ib), C.byref(ir))
    return ib.value, ir.value


def gammainc(a, x):
    return lib().co3o_gammainc(a, x)


def model_weights(E, M, ibeta, ir):
    w = np.zeros(1 << (1 + E + M), np.uint32)
    rc = lib().co3o_model_weights(E, M, ibeta, ir, w)
    if rc != OK:
        raise ValueError("co3o_model_weights: bad arguments")
    return w


def huffman(w):
    w = np.ascontiguousarray(w, np.uint32)
    ln = np.zeros(len(w), np.uint8)
    f = C.c_uint32()
    rc = lib().co3o_huffman(w, len(w), ln, C.byref(f))
    if rc != OK:
        raise ValueError("co3o_huffman: bad arguments")
    return ln, int(f.value)


def huffman_counts(counts):
    c = np.ascontiguousarray(counts, np.uint64)
    ln = np.zeros(len(c), np.uint8)
    f = C.c_uint32()
    rc = lib().co3o_huffman_counts(c, len(c), ln, C.byref(f))
    if rc != OK:
        raise ValueError("co3o_huffman_counts: bad arguments")
    return ln, int(f.value)


def canonical(ln):
    ln = np.ascontiguousarray(ln, np.uint8)
    code = np.zeros(len(ln), np.uint32)
    lib().co3o_canonical(ln, len(ln), code)
    return code


class Partition:
    """Static cut of a user's row into chunks and sub-chunks (see the container comment in C)."""

    def __init__(self, d, seg_offsets):
        off = np.ascontiguousarray(seg_offsets, np.int64)
        S = len(off) - 1
        ns = _i64()
        nc = lib().co3o_partition(d, S, off, None, None, None, None, C.byref(ns))
        if nc < 0:
            raise ValueError("bad segment offsets")
        self.d, self.S, self.off = int(d), S, off
        self.n_chunks, self.n_sub = int(nc), int(ns.value)
        self.chunk_seg = np.zeros(max(nc, 1), np.int32)
        self.chunk_start = np.zeros(max(nc, 1), np.int64)
        self.chunk_end = np.zeros(max(nc, 1), np.int64)
        self.sub_base = np.zeros(max(nc, 1), np.int64)
        lib().co3o_partition(d, S, off, self.chunk_seg.ctypes.data, self.chunk_start.ctypes.data,
                             self.chunk_end.ctypes.data, self.sub_base.ctypes.data, C.byref(ns))


def encode_user(sym_row, part, nsym, lens, codes, cap_words):
    payload = np.zeros(max(cap_words, 1), np.uint32)
    sub_bits = np.zeros(max(part.n_sub, 1), np.uint16)
    chunk_off = np.zeros(part.n_chunks + 1, np.uint32)
    ub = C.c_uint64()
    rc = lib().co3o_encode_user(np.ascontiguousarray(sym_row), part.n_chunks, part.chunk_seg,
                                part.chunk_start, part.chunk_end, part.sub_base, nsym,
                                np.ascontiguousarray(lens, np.uint8),
                                np.ascontiguousarray(codes, np.uint32),
                                payload, cap_words, sub_bits, chunk_off, C.byref(ub))
    return rc, payload, sub_bits, chunk_off, int(ub.value)


def decode_aggregate(payload, sub_bits, chunk_off, part, hdr, E, M, want_symbols=False, lens=None):
    """payload [U][cap], sub_bits [U][n_sub], chunk_off [U][n_chunks+1], hdr [S][3] int32;
    lens [S][2^B] u8: the code lengths, when they are side information (empirical-histogram code)."""
    U, cap = payload.shape
    avg = np.zeros(part.d, np.float32)
    sym = np.zeros((U, part.d), np.uint8) if want_symbols else None
    rc = lib().co3o_decode_aggregate(
        np.ascontiguousarray(payload), cap, np.ascontiguousarray(sub_bits), sub_bits.shape[1],
        np.ascontiguousarray(chunk_off), U, part.n_chunks, part.chunk_seg, part.chunk_start,
        part.chunk_end, part.sub_base, part.S, np.ascontiguousarray(hdr, np.int32), E, M, avg,
        sym.ctypes.data if want_symbols else None, part.d,
        None if lens is None else np.ascontiguousarray(lens, np.uint8).ctypes.data)
    return rc, avg, sym


class IterationResult:
    pass


class OracleCO3:
    """Carries the method's state across iterations and runs one iteration at a time.

    encode(g, m): g [U][ld] fp32 gradients, m [U][ld] fp32 memory (updated in place).
    """

    def __init__(self, d, n_users, E, M, seg_offsets=None, gamma=0.9, mode=MODE_LAGGED,
                 cap_words=None, rule=RULE_POLY):
        self.d, self.U, self.E, self.M = int(d), int(n_users), int(E), int(M)
        self.nsym = 1 << (1 + E + M)
        off = [0, d] if seg_offsets is None else list(seg_offsets)
        self.part = Partition(d, off)
        self.S = self.part.S
        self.gamma = float(np.float32(gamma))
        self.mode = mode
        self.rule = rule
        self.t = 0
        self.bias_next = np.zeros(self.S, np.int32)
        self.hdr_next = np.zeros((self.S, 3), np.int32)   # MODE_LAGGED_CODE: header of the coming iteration
        # worst case: 16 bits per symbol, every chunk padded to 128 bits
        worst = sum(4 * ((16 * int(e - s) + 127) // 128)
                    for s, e in zip(self.part.chunk_start[:self.part.n_chunks],
                                    self.part.chunk_end[:self.part.n_chunks]))
        self.worst_case_words = worst
        self.cap_words = worst if cap_words is None else int(cap_words)

    def encode(self, g, m):
        U, S, E, M, off = self.U, self.S, self.E, self.M, self.part.off
        assert g.shape == m.shape and g.shape[0] == U and g.dtype == np.float32
        r = IterationResult()
        bias_t = np.zeros(S, np.int32)
        if self.t == 0 or self.mode == MODE_CURRENT:
            for l in range(S):
                N, S1, S2, _ = stats(g, m, int(off[l]), int(off[l + 1]), self.gamma)
                be, al = fit(N, S1, S2)
                bias_t[l] = bias_by_rule(self.rule, be, al, E, M)
        else:
            bias_t[:] = self.bias_next
        sym = np.zeros((U, self.d), np.uint8)
        hist = np.zeros((S, self.nsym), np.uint64)
        r.fit = np.zeros((S, 2))
        r.moments = np.zeros((S, 3))
        r.nonfinite = 0
        hdr = np.zeros((S, 3), np.int32)
        for l in range(S):
            N, S1, S2, nf = convert(g, m, sym, int(off[l]), int(off[l + 1]), self.gamma, E, M,
                                    int(bias_t[l]), hist[l])
            be, al = fit(N, S1, S2)
            self.bias_next[l] = bias_by_rule(self.rule, be, al, E, M)
            if self.mode == MODE_LAGGED_CODE and self.t > 0:
                hdr[l] = self.hdr_next[l]              # fixed by iteration t-1 (its bias is bias_t[l])
            else:
                ib, ir = header(be, al, int(bias_t[l]))
                hdr[l] = (bias_t[l], ib, ir)
            # the header the coming iteration would use: this fit, relative to the coming bias
            ibn, irn = header(be, al, int(self.bias_next[l]))
            self.hdr_next[l] = (self.bias_next[l], ibn, irn)
            r.fit[l] = (be, al)
            r.moments[l] = (N, S1, S2)
            r.nonfinite += nf
        lens = np.zeros((S, self.nsym), np.uint8)
        codes = np.zeros((S, self.nsym), np.uint32)
        r.floor = np.zeros(S, np.int64)
        for l in range(S):
            if self.mode == MODE_EMPIRICAL:
                lens[l], r.floor[l] = huffman_counts(hist[l])
            else:
                w = model_weights(E, M, int(hdr[l, 1]), int(hdr[l, 2]))
                lens[l], r.floor[l] = huffman(w)
            codes[l] = canonical(lens[l])
        cap = self.cap_words
        r.payload = np.zeros((U, max(cap, 1)), np.uint32)
        r.sub_bits = np.zeros((U, max(self.part.n_sub, 1)), np.uint16)
        r.chunk_off = np.zeros((U, self.part.n_chunks + 1), np.uint32)
        r.user_bits = np.zeros(U, np.uint64)
        r.status = OK
        for u in range(U):
            rc, p, sb, co, ub = encode_user(sym[u], self.part, self.nsym, lens, codes, cap)
            if rc != OK:
                r.status = rc
            r.payload[u, :len(p)] = p
            r.sub_bits[u], r.chunk_off[u], r.user_bits[u] = sb, co, ub
        r.sym, r.hist, r.hdr, r.lens, r.codes, r.bias = sym, hist, hdr, lens, codes, bias_t
        self.t += 1
        return r

    def decode_aggregate_update(self, payload, sub_bits, chunk_off, hdr, weights, step):
        """Algorithm 1 lines 13-14 with the model update: w <- fl32(w + fl32(step * avg)), in place.
        The caller passes the signed step (the paper writes the update with both signs)."""
        rc, avg, _ = self.decode_aggregate(payload, sub_bits, chunk_off, hdr)
        if rc == OK:
            weights += (np.float32(step) * avg).astype(np.float32)
        return rc, avg

    def decode_aggregate(self, payload, sub_bits, chunk_off, hdr, want_symbols=False, lens=None):
        return decode_aggregate(payload, sub_bits, chunk_off, self.part, hdr, self.E, self.M,
                                want_symbols, lens)
