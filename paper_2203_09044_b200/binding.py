"""ctypes binding of the CO3 CUDA library (include/co3.h): argument marshalling only.

Every step of the pipeline runs in the library's CUDA kernels.  There is no CPU fallback: if the
library has not been built (python -m paper_2203_09044_b200.build, or __graft_entry__.build())
loading raises.  torch is used for device memory and streams only.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libco3.so")

OK, EINVAL, ENOMEM, ECUDA, ECAPACITY, ECORRUPT, ENONFINITE = 0, -1, -2, -3, -4, -5, -6
FLAG_CAPACITY, FLAG_CORRUPT, FLAG_NONFINITE = 1, 2, 4
BIAS_CURRENT, BIAS_LAGGED, CODE_LAGGED, CODE_EMPIRICAL = 0, 1, 2, 3
RULE_POLY, RULE_OPT = 0, 1
FLAG_TIMEOUT = 8
FLAG_INEXACT = 16

EXPORTS = [
    "co3_plan_create", "co3_plan_destroy", "co3_sizes", "co3_encode", "co3_decode_aggregate",
    "co3_iteration_host", "co3_status", "co3_get_fit", "co3_state_export", "co3_state_import",
    "co3_debug_symbols", "co3_debug_hist", "co3_debug_code", "co3_model_weights", "co3_partition",
    "co3_strerror", "co3_profile_enable", "co3_profile_collect", "co3_launch_count",
    "co3_moments_static", "co3_state_header", "co3_decode_aggregate_update",
    "co3_bias_opt_table", "co3_grid_distortion", "co3_encode_empirical", "co3_decode_aggregate_empirical",
    "co3_profile_stride", "co3_tiled_begin", "co3_tiled_statistics", "co3_tiled_convert", "co3_tiled_finish",
    "co3_moments_export", "co3_moments_import", "co3_set_fit_override", "co3_debug_encode_stalled",
    "co3_model_checksum", "co3_balanced_split",
]
ELIMIT = -7
STATIC_MAX_ELEMENTS = 1 << 29

KERNEL_NAMES = ["stats", "fit", "convert", "code_enc", "reconvert", "enc_scan", "enc_pack", "code_dec",
                "decode"]


class Format(C.Structure):
    _fields_ = [("exp_bits", C.c_int32), ("mant_bits", C.c_int32)]


class Config(C.Structure):
    _fields_ = [("d", C.c_int64), ("ld", C.c_int64), ("n_users", C.c_int32), ("fmt", Format),
                ("n_segments", C.c_int32), ("seg_offsets", C.POINTER(C.c_int64)),
                ("gamma", C.c_float), ("bias_mode", C.c_int32), ("cap_words", C.c_int64),
                ("bias_rule", C.c_int32), ("reserved", C.c_int32)]


HDR_DTYPE = np.dtype([("bias", np.int8), ("ibeta", np.int8), ("ir", np.int16)])

_lib = None


class Co3Error(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib().co3_strerror(code).decode()} ({code})")


def lib():
    """Load csrc/libco3.so; raises if it is missing (there is no other implementation)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not built: run `python -m paper_2203_09044_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, i64p = C.c_void_p, C.POINTER(C.c_int64)
    L.co3_plan_create.restype = C.c_int
    L.co3_plan_create.argtypes = [C.POINTER(vp), C.POINTER(Config)]
    L.co3_plan_destroy.restype = None
    L.co3_plan_destroy.argtypes = [vp]
    L.co3_sizes.restype = C.c_int
    L.co3_sizes.argtypes = [vp, i64p, i64p, i64p]
    L.co3_encode.restype = C.c_int
    L.co3_encode.argtypes = [vp] * 9
    L.co3_decode_aggregate.restype = C.c_int
    L.co3_decode_aggregate.argtypes = [vp] * 7
    L.co3_encode_empirical.restype = C.c_int
    L.co3_encode_empirical.argtypes = [vp] * 10
    L.co3_decode_aggregate_empirical.restype = C.c_int
    L.co3_decode_aggregate_empirical.argtypes = [vp] * 8
    L.co3_decode_aggregate_update.restype = C.c_int
    L.co3_decode_aggregate_update.argtypes = [vp] * 7 + [C.c_float, vp]
    L.co3_iteration_host.restype = C.c_int
    L.co3_iteration_host.argtypes = [vp] * 12
    L.co3_status.restype = C.c_int
    L.co3_status.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_uint64), C.c_int32]
    L.co3_get_fit.restype = C.c_int
    L.co3_get_fit.argtypes = [vp, C.c_int32] + [C.POINTER(C.c_double)] * 5
    L.co3_state_export.restype = C.c_int
    L.co3_state_export.argtypes = [vp, i64p, vp]
    L.co3_state_import.restype = C.c_int
    L.co3_state_import.argtypes = [vp, C.c_int64, vp]
    L.co3_debug_symbols.restype = C.c_int
    L.co3_debug_symbols.argtypes = [vp, vp, vp]
    L.co3_debug_hist.restype = C.c_int
    L.co3_debug_hist.argtypes = [vp, vp]
    L.co3_debug_code.restype = C.c_int
    L.co3_debug_code.argtypes = [vp, vp, vp, vp]
    L.co3_model_weights.restype = C.c_int
    L.co3_model_weights.argtypes = [Format, C.c_int32, C.c_int32, vp]
    L.co3_partition.restype = C.c_int64
    L.co3_partition.argtypes = [C.c_int64, C.c_int32, vp, vp, vp, vp, vp, i64p]
    L.co3_profile_enable.restype = C.c_int
    L.co3_profile_enable.argtypes = [vp, C.c_uint32, C.c_int32]
    L.co3_tiled_begin.restype = C.c_int
    L.co3_tiled_begin.argtypes = [vp, C.POINTER(C.c_int32)]
    L.co3_tiled_statistics.restype = C.c_int
    L.co3_tiled_statistics.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, vp]
    L.co3_tiled_convert.restype = C.c_int
    L.co3_tiled_convert.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, vp]
    L.co3_tiled_finish.restype = C.c_int
    L.co3_tiled_finish.argtypes = [vp] * 7
    L.co3_moments_export.restype = C.c_int
    L.co3_moments_export.argtypes = [vp, vp, vp]
    L.co3_moments_import.restype = C.c_int
    L.co3_moments_import.argtypes = [vp, vp, vp]
    L.co3_profile_stride.restype = C.c_int
    L.co3_profile_stride.argtypes = [vp, C.c_int32]
    L.co3_profile_collect.restype = C.c_int
    L.co3_profile_collect.argtypes = [vp, vp, vp]
    L.co3_launch_count.restype = C.c_int64
    L.co3_launch_count.argtypes = [vp]
    L.co3_moments_static.restype = C.c_int
    L.co3_moments_static.argtypes = [vp, vp, C.c_int64, C.c_float, vp, vp]
    L.co3_state_header.restype = C.c_int
    L.co3_state_header.argtypes = [vp, C.c_int32, vp]
    L.co3_bias_opt_table.restype = C.c_int
    L.co3_bias_opt_table.argtypes = [Format, vp]
    L.co3_grid_distortion.restype = C.c_double
    L.co3_grid_distortion.argtypes = [Format, C.c_int32, C.c_int32]
    L.co3_set_fit_override.restype = C.c_int
    L.co3_set_fit_override.argtypes = [vp, vp]
    L.co3_debug_encode_stalled.restype = C.c_int
    L.co3_debug_encode_stalled.argtypes = [vp] * 6 + [C.c_int32, vp]
    L.co3_model_checksum.restype = C.c_uint64
    L.co3_model_checksum.argtypes = [Format]
    L.co3_balanced_split.restype = C.c_int
    L.co3_balanced_split.argtypes = [vp, vp, C.c_int64, C.c_int32, C.c_int32, vp]
    L.co3_strerror.restype = C.c_char_p
    L.co3_strerror.argtypes = [C.c_int]
    _lib = L
    return L


def model_weights(exp_bits, mant_bits, ibeta, ir):
    """Host only: integer model weights per symbol byte for header indices (ibeta, ir)."""
    w = np.zeros(1 << (1 + exp_bits + mant_bits), np.uint32)
    rc = lib().co3_model_weights(Format(exp_bits, mant_bits), ibeta, ir, w.ctypes.data)
    if rc != OK:
        raise Co3Error(rc, "co3_model_weights")
    return w


def model_checksum(exp_bits, mant_bits):
    """Host only: digest of the whole model-weight table of a format (0: unsupported format)."""
    return int(lib().co3_model_checksum(Format(exp_bits, mant_bits)))


def balanced_split(cost, seg, teams, max_blocks):
    """Host only: cuts (max_blocks + 1 int32) and the number of blocks in use (co3_balanced_split)."""
    c = np.ascontiguousarray(cost, np.float64)
    g = np.ascontiguousarray(seg, np.int32)
    part = np.zeros(max_blocks + 1, np.int32)
    nb = lib().co3_balanced_split(c.ctypes.data, g.ctypes.data, len(c), int(teams), int(max_blocks), part.ctypes.data)
    if nb < 0:
        raise Co3Error(EINVAL, "co3_balanced_split")
    return part, nb


def bias_opt_table(exp_bits, mant_bits):
    """[23][8] int16 table behind RULE_OPT (host only)."""
    tab = np.zeros((23, 8), np.int16)
    rc = lib().co3_bias_opt_table(Format(exp_bits, mant_bits), tab.ctypes.data)
    if rc != OK:
        raise Co3Error(rc, "co3_bias_opt_table")
    return tab


def grid_distortion(exp_bits, mant_bits, ibeta, ir):
    return float(lib().co3_grid_distortion(Format(exp_bits, mant_bits), int(ibeta), int(ir)))


def partition(d, seg_offsets):
    """Host only: (chunk_seg, chunk_start, chunk_end, sub_base, n_sub) of the static partition."""
    off = np.ascontiguousarray(seg_offsets, np.int64)
    ns = C.c_int64()
    nc = lib().co3_partition(d, len(off) - 1, off.ctypes.data, None, None, None, None, C.byref(ns))
    if nc < 0:
        raise Co3Error(int(nc), "co3_partition")
    seg = np.zeros(nc, np.int32)
    st, en, sb = (np.zeros(nc, np.int64) for _ in range(3))
    lib().co3_partition(d, len(off) - 1, off.ctypes.data, seg.ctypes.data, st.ctypes.data,
                        en.ctypes.data, sb.ctypes.data, C.byref(ns))
    return seg, st, en, sb, int(ns.value)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def moments_static(grad, residual, n, gamma, moments, stream=None):
    """co3_moments_static: N, sum|a|, sum a^2, non-finite count of a = g + gamma m over n elements
    into `moments` (4 float64 on the device), with no allocation inside the library.  Returns the
    C return code (0, or a negative CO3_E* value such as ELIMIT)."""
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return int(lib().co3_moments_static(_ptr(grad), _ptr(residual), int(n), float(gamma), _ptr(moments),
                                        C.c_void_p(s.cuda_stream)))


class Plan:
    """co3_plan plus the torch buffers of one pipeline instance on the current CUDA device."""

    def __init__(self, d, n_users, exp_bits, mant_bits, seg_offsets=None, gamma=0.9,
                 bias_mode=BIAS_LAGGED, cap_words=None, ld=None, bias_rule=RULE_POLY):
        import torch
        self.torch = torch
        L = lib()
        self.d, self.U, self.E, self.M = int(d), int(n_users), int(exp_bits), int(mant_bits)
        self.ld = int(ld) if ld is not None else (self.d + 3) // 4 * 4
        self.nsym = 1 << (1 + self.E + self.M)
        self.bias_mode = int(bias_mode)
        off = np.ascontiguousarray([0, d] if seg_offsets is None else seg_offsets, np.int64)
        self.S = len(off) - 1
        self._off = off
        # worst case needs the partition; compute it on the host first
        _, st, en, _, _ = partition(self.d, off)
        worst = int(sum(4 * ((16 * int(e - s) + 127) // 128) for s, e in zip(st, en)))
        self.cap_words = int(cap_words) if cap_words is not None else worst
        cfg = Config(self.d, self.ld, self.U, Format(self.E, self.M), self.S,
                     off.ctypes.data_as(C.POINTER(C.c_int64)), float(gamma), int(bias_mode),
                     self.cap_words, int(bias_rule), 0)
        h = C.c_void_p()
        rc = L.co3_plan_create(C.byref(h), C.byref(cfg))
        if rc != OK:
            raise Co3Error(rc, "co3_plan_create")
        self.handle = h
        nc, ns, wc = C.c_int64(), C.c_int64(), C.c_int64()
        L.co3_sizes(h, C.byref(nc), C.byref(ns), C.byref(wc))
        self.n_chunks, self.n_sub, self.worst_case_words = nc.value, ns.value, wc.value

    def close(self):
        if getattr(self, "handle", None):
            lib().co3_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- buffers ---------------------------------------------------------------------------
    def alloc_outputs(self, device="cuda"):
        t = self.torch
        return dict(
            bitstream=t.zeros((self.U, self.cap_words), dtype=t.int32, device=device),
            sub_bits=t.zeros((self.U, max(self.n_sub, 1)), dtype=t.int16, device=device),
            chunk_off=t.zeros((self.U, self.n_chunks + 1), dtype=t.int32, device=device),
            user_bits=t.zeros((self.U,), dtype=t.int64, device=device),
            hdr=t.zeros((self.S,), dtype=t.int32, device=device),
            avg=t.zeros((self.d,), dtype=t.float32, device=device),
            code_lens=t.zeros((self.S, self.nsym), dtype=t.uint8, device=device),   # CODE_EMPIRICAL only
        )

    def _stream(self, stream):
        s = self.torch.cuda.current_stream() if stream is None else stream
        return C.c_void_p(s.cuda_stream)

    # ---- the C-ABI calls -------------------------------------------------------------------
    def encode(self, grad, residual, out, stream=None):
        if self.bias_mode == CODE_EMPIRICAL:
            rc = lib().co3_encode_empirical(self.handle, _ptr(grad), _ptr(residual), _ptr(out["bitstream"]),
                                            _ptr(out["sub_bits"]), _ptr(out["chunk_off"]), _ptr(out["user_bits"]),
                                            _ptr(out["hdr"]), _ptr(out["code_lens"]), self._stream(stream))
        else:
            rc = lib().co3_encode(self.handle, _ptr(grad), _ptr(residual), _ptr(out["bitstream"]),
                                  _ptr(out["sub_bits"]), _ptr(out["chunk_off"]), _ptr(out["user_bits"]),
                                  _ptr(out["hdr"]), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_encode")

    def encode_tiled(self, tile_users, make_tile, residual, out, stream=None, around_call=None):
        """One iteration with the gradient supplied tile by tile: make_tile(user0, n) returns the
        [n][ld] fp32 cuda gradient of users user0 .. user0 + n - 1 (it may reuse one buffer: each tile
        is consumed by kernels enqueued on the stream before the next make_tile call returns work on
        that same stream).  Bit for bit the result of encode() on the whole gradient.
        around_call(False) / around_call(True), if given, run right before / after every library call
        (a timing hook: whatever make_tile does stays outside)."""
        need = C.c_int32()
        rc = lib().co3_tiled_begin(self.handle, C.byref(need))
        if rc != OK:
            raise Co3Error(rc, "co3_tiled_begin")
        passes = (["co3_tiled_statistics"] if need.value else []) + ["co3_tiled_convert"]
        for name in passes:
            for u0 in range(0, self.U, tile_users):
                n = min(tile_users, self.U - u0)
                g = make_tile(u0, n)
                if around_call:
                    around_call(False)
                rc = getattr(lib(), name)(self.handle, _ptr(g), _ptr(residual), u0, n, self._stream(stream))
                if around_call:
                    around_call(True)
                if rc != OK:
                    raise Co3Error(rc, name)
        if around_call:
            around_call(False)
        rc = lib().co3_tiled_finish(self.handle, _ptr(out["bitstream"]), _ptr(out["sub_bits"]), _ptr(out["chunk_off"]),
                                    _ptr(out["user_bits"]), _ptr(out["hdr"]), self._stream(stream))
        if around_call:
            around_call(True)
        if rc != OK:
            raise Co3Error(rc, "co3_tiled_finish")

    # The phases of a tiled iteration one by one (encode_tiled strings them together); between them a
    # caller may pool the moments of several plans (moments_export / moments_import).
    def tiled_begin(self):
        """Start a tiled iteration; True if statistics tiles have to come before the convert tiles."""
        need = C.c_int32()
        rc = lib().co3_tiled_begin(self.handle, C.byref(need))
        if rc != OK:
            raise Co3Error(rc, "co3_tiled_begin")
        return bool(need.value)

    def tiled_statistics(self, grad_tile, residual, user0, n_users, stream=None):
        rc = lib().co3_tiled_statistics(self.handle, _ptr(grad_tile), _ptr(residual), user0, n_users, self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_tiled_statistics")

    def tiled_convert(self, grad_tile, residual, user0, n_users, stream=None):
        rc = lib().co3_tiled_convert(self.handle, _ptr(grad_tile), _ptr(residual), user0, n_users, self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_tiled_convert")

    def tiled_finish(self, out, stream=None):
        rc = lib().co3_tiled_finish(self.handle, _ptr(out["bitstream"]), _ptr(out["sub_bits"]), _ptr(out["chunk_off"]),
                                    _ptr(out["user_bits"]), _ptr(out["hdr"]), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_tiled_finish")

    def moments_export(self, moments=None, stream=None):
        """[S][3] fp64 cuda: (finite entries, sum |a|, sum a^2) of every segment, all users pooled."""
        import torch
        if moments is None:
            moments = torch.empty((self.S, 3), dtype=torch.float64, device="cuda")
        rc = lib().co3_moments_export(self.handle, _ptr(moments), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_moments_export")
        return moments

    def moments_import(self, moments, stream=None):
        """The sums the next fit uses instead of the plan's own ([S][3] fp64 cuda, contiguous)."""
        assert moments.is_cuda and moments.is_contiguous() and tuple(moments.shape) == (self.S, 3)
        rc = lib().co3_moments_import(self.handle, _ptr(moments), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_moments_import")

    def decode_aggregate(self, out, avg=None, stream=None):
        avg = out["avg"] if avg is None else avg
        if self.bias_mode == CODE_EMPIRICAL:
            rc = lib().co3_decode_aggregate_empirical(self.handle, _ptr(out["bitstream"]), _ptr(out["sub_bits"]),
                                                      _ptr(out["chunk_off"]), _ptr(out["hdr"]),
                                                      _ptr(out["code_lens"]), _ptr(avg), self._stream(stream))
        else:
            rc = lib().co3_decode_aggregate(self.handle, _ptr(out["bitstream"]), _ptr(out["sub_bits"]),
                                            _ptr(out["chunk_off"]), _ptr(out["hdr"]), _ptr(avg),
                                            self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_decode_aggregate")
        return avg

    def decode_aggregate_update(self, out, weights, step, avg=None, stream=None):
        """decode_aggregate with w <- w + step * avg fused in (weights: [d] fp32 cuda tensor, in place)."""
        avg = out["avg"] if avg is None else avg
        rc = lib().co3_decode_aggregate_update(self.handle, _ptr(out["bitstream"]), _ptr(out["sub_bits"]),
                                               _ptr(out["chunk_off"]), _ptr(out["hdr"]), _ptr(avg),
                                               _ptr(weights), C.c_float(float(step)), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_decode_aggregate_update")
        return avg

    def iteration_host(self, h_grad, d_grad, residual, out, h_avg, stream=None):
        rc = lib().co3_iteration_host(self.handle, _ptr(h_grad), _ptr(d_grad), _ptr(residual),
                                      _ptr(out["bitstream"]), _ptr(out["sub_bits"]),
                                      _ptr(out["chunk_off"]), _ptr(out["user_bits"]), _ptr(out["hdr"]),
                                      _ptr(out["avg"]), _ptr(h_avg), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_iteration_host")

    def status(self, clear=False):
        f, n = C.c_uint32(), C.c_uint64()
        rc = lib().co3_status(self.handle, C.byref(f), C.byref(n), int(clear))
        if rc != OK:
            raise Co3Error(rc, "co3_status")
        return int(f.value), int(n.value)

    def get_fit(self, seg):
        v = [C.c_double() for _ in range(5)]
        rc = lib().co3_get_fit(self.handle, seg, *[C.byref(x) for x in v])
        if rc != OK:
            raise Co3Error(rc, "co3_get_fit")
        return tuple(x.value for x in v)        # beta, alpha, N, S1, S2

    def set_fit_override(self, fit=None):
        """Test hook: every later fit takes (beta, alpha) per segment from `fit` ([S][2] float64);
        None switches it off."""
        if fit is None:
            rc = lib().co3_set_fit_override(self.handle, None)
        else:
            f = np.ascontiguousarray(fit, np.float64)
            assert f.shape == (self.S, 2)
            rc = lib().co3_set_fit_override(self.handle, f.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_set_fit_override")

    def debug_encode_stalled(self, out, spin_limit=1000, stream=None):
        """Test hook: the packing kernel once more with the block of (user 0, chunk 0) left out, so that
        the bounded waits for that chunk's size run out after spin_limit polls (FLAG_TIMEOUT)."""
        rc = lib().co3_debug_encode_stalled(self.handle, _ptr(out["bitstream"]), _ptr(out["sub_bits"]),
                                            _ptr(out["chunk_off"]), _ptr(out["user_bits"]), _ptr(out["hdr"]),
                                            int(spin_limit), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_debug_encode_stalled")

    def state_export(self):
        it = C.c_int64()
        nb = np.zeros(self.S, np.int32)
        rc = lib().co3_state_export(self.handle, C.byref(it), nb.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_state_export")
        return int(it.value), nb

    def state_import(self, iteration, next_bias):
        nb = np.ascontiguousarray(next_bias, np.int32)
        rc = lib().co3_state_import(self.handle, int(iteration), nb.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_state_import")

    def state_header(self, next_header=None):
        """CODE_LAGGED only: the header of the coming iteration, as an [S][3] int32 array
        (bias, ibeta, ir).  With an argument it is imported instead."""
        raw = np.zeros(self.S, np.int32)
        if next_header is not None:
            h = np.ascontiguousarray(next_header, np.int32)
            raw = ((h[:, 0] & 0xFF) | ((h[:, 1] & 0xFF) << 8) | ((h[:, 2] & 0xFFFF) << 16)).astype(np.uint32).view(np.int32)
            raw = np.ascontiguousarray(raw)
        rc = lib().co3_state_header(self.handle, 0 if next_header is None else 1, raw.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_state_header")
        v = raw.view(np.uint32)
        out = np.zeros((self.S, 3), np.int32)
        out[:, 0] = (v & 0xFF).astype(np.uint8).view(np.int8)
        out[:, 1] = ((v >> 8) & 0xFF).astype(np.uint8).view(np.int8)
        out[:, 2] = ((v >> 16) & 0xFFFF).astype(np.uint16).view(np.int16)
        return out

    def profile_enable(self, kernel_names=None, max_records=4096):
        """Trace the named kernel classes (all if None; [] switches tracing off)."""
        names = KERNEL_NAMES if kernel_names is None else kernel_names
        mask = 0
        for n in names:
            mask |= 1 << KERNEL_NAMES.index(n)
        rc = lib().co3_profile_enable(self.handle, mask, max_records)
        if rc != OK:
            raise Co3Error(rc, "co3_profile_enable")

    def profile_stride(self, every):
        """Time only every `every`-th launch of each traced kernel class."""
        rc = lib().co3_profile_stride(self.handle, int(every))
        if rc != OK:
            raise Co3Error(rc, "co3_profile_stride")

    def profile_collect(self):
        """{kernel class: (total ms, launches)} since the last collect (synchronises)."""
        ms = np.zeros(len(KERNEL_NAMES), np.float64)
        n = np.zeros(len(KERNEL_NAMES), np.int64)
        rc = lib().co3_profile_collect(self.handle, ms.ctypes.data, n.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_profile_collect")
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_NAMES)}

    def launch_count(self):
        return int(lib().co3_launch_count(self.handle))

    def debug_symbols(self, stream=None):
        t = self.torch
        sym = t.zeros((self.U, self.d), dtype=t.uint8, device="cuda")
        rc = lib().co3_debug_symbols(self.handle, _ptr(sym), self._stream(stream))
        if rc != OK:
            raise Co3Error(rc, "co3_debug_symbols")
        return sym

    def debug_hist(self):
        h = np.zeros((self.S, self.nsym), np.uint64)
        rc = lib().co3_debug_hist(self.handle, h.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_debug_hist")
        return h

    def debug_code(self, hdr):
        ln = np.zeros((self.S, self.nsym), np.uint8)
        cw = np.zeros((self.S, self.nsym), np.uint32)
        rc = lib().co3_debug_code(self.handle, _ptr(hdr), ln.ctypes.data, cw.ctypes.data)
        if rc != OK:
            raise Co3Error(rc, "co3_debug_code")
        return ln, cw


def hdr_to_numpy(hdr_tensor):
    """[S] int32 device tensor of packed headers -> [S][3] int32 (bias, ibeta, ir)."""
    raw = hdr_tensor.cpu().numpy().view(HDR_DTYPE)
    return np.stack([raw["bias"].astype(np.int32), raw["ibeta"].astype(np.int32),
                     raw["ir"].astype(np.int32)], axis=1)


def hdr_from_numpy(hdr3, device="cuda"):
    import torch
    raw = np.zeros(len(hdr3), HDR_DTYPE)
    raw["bias"], raw["ibeta"], raw["ir"] = hdr3[:, 0], hdr3[:, 1], hdr3[:, 2]
    return torch.from_numpy(raw.view(np.int32).copy()).to(device)
