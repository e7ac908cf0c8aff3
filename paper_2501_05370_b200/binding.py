"""Thin ctypes binding of libsds (include/sds.h). Argument marshalling only: every step of the
window runs in the library's CUDA kernels. PyTorch provides device memory and streams.

There is no CPU fallback: importing works without a GPU (so that symbols can be inspected), but
constructing a Sampler without CUDA raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

from . import build as _build

# ---- constants mirrored from sds.h ----
SDS_OK = 0
SDS_EINVAL, SDS_ESTATE, SDS_ENOMEM, SDS_EUNSUPPORTED = -1, -2, -3, -4
SDS_ECUDA, SDS_ETIMEOUT, SDS_ENONFINITE, SDS_ECALLBACK = -5, -6, -7, -8
SDS_DEN_GMM, SDS_DEN_MLP, SDS_DEN_CALLBACK, SDS_DEN_PHI4 = 1, 2, 3, 4
SDS_F32, SDS_BF16 = 0, 1
SDS_FROZEN_PREV, SDS_FROZEN_EXACT, SDS_INDEPENDENT, SDS_PICARD = 0, 1, 2, 3
(GET_X, GET_TAIL, GET_DQ, GET_DC, GET_Y, GET_N, GET_ACT, GET_ROWOFF, GET_S1, GET_S2, GET_ELL, GET_LOGU,
 GET_ACCMASK, GET_JSTAR, GET_NFE_CALLS, GET_NFE_ROWS, GET_CTL, GET_ROWK, GET_DP) = range(1, 20)

DENOISE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p)


class SdsSchedule(C.Structure):
    _fields_ = [("K", C.c_int32), ("a", C.c_void_p), ("c", C.c_void_p), ("sigma", C.c_void_p),
                ("tcond", C.c_void_p), ("tcond_dim", C.c_int32)]


class SdsDenoiser(C.Structure):
    _fields_ = [("kind", C.c_int32), ("ncomp", C.c_int32), ("means_dev", C.c_void_p), ("logw_dev", C.c_void_p),
                ("means_dtype", C.c_int32), ("nlayer", C.c_int32), ("W_dev", C.c_void_p), ("bias_dev", C.c_void_p),
                ("temb_dev", C.c_void_p), ("dims", C.c_void_p), ("fn", DENOISE_FN), ("user", C.c_void_p),
                ("grid_side", C.c_int32), ("coupling", C.c_float), ("periodic", C.c_int32)]


EXPORTS = {
    "sds_workspace_bytes": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]),
    "sds_create": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.POINTER(C.c_void_p)]),
    "sds_workspace_bytes_with_drafter": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32,
                                                   C.c_int32, C.POINTER(C.c_size_t)]),
    "sds_create_with_drafter": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                                          C.POINTER(C.c_void_p)]),
    "sds_workspace_bytes_picard": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                                             C.POINTER(C.c_size_t)]),
    "sds_create_picard": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32,
                                    C.c_int32, C.POINTER(C.c_void_p)]),
    "sds_bind": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_uint64, C.c_int32, C.c_int64]),
    "sds_reset": (C.c_int, [C.c_void_p]),
    "sds_draft": (C.c_int, [C.c_void_p]),
    "sds_verify_window": (C.c_int, [C.c_void_p]),
    "sds_advance": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64)]),
    "sds_sample_all": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "sds_sample_all_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "sds_get": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_int32]),
    "sds_set_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "sds_denoise": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "sds_rng_normals": (C.c_int, [C.c_uint64, C.c_int32, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "sds_rng_uniforms": (C.c_int, [C.c_uint64, C.c_int64, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p]),
    "sds_selftest_bounded_wait": (C.c_int, [C.c_int32, C.c_void_p, C.c_void_p]),
    "sds_launch_count": (C.c_int64, [C.c_void_p]),
    "sds_set_option": (C.c_int, [C.c_void_p, C.c_int32, C.c_int64]),
    "sds_set_temperature": (C.c_int, [C.c_void_p, C.c_double]),
    "sds_set_projection": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32]),
    "sds_profile": (C.c_int, [C.c_void_p, C.c_int32]),
    "sds_profile_read": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]),
    "sds_gmm_denoise_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "sds_strerror": (C.c_char_p, [C.c_int]),
    "sds_last_cuda_error": (C.c_int, [C.c_void_p]),
    "sds_destroy": (None, [C.c_void_p]),
}

_lib = None


def lib_path() -> str:
    return _build.LIB


def load() -> C.CDLL:
    """Load libsds.so (building it with nvcc first if the sources are newer). Raises if neither the
    library nor a compiler is available: there is no other implementation to fall back to."""
    global _lib
    if _lib is not None:
        return _lib
    if _build.needs_build():
        _build.build()
    if not os.path.exists(_build.LIB):
        raise RuntimeError("libsds.so is missing and could not be built")
    lib = C.CDLL(_build.LIB)
    for name, (res, args) in EXPORTS.items():
        fn = getattr(lib, name)          # AttributeError if an export is missing
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


class SdsError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        msg = load().sds_strerror(code).decode()
        super().__init__(f"{where}: {msg} (code {code}" + (f", cuda error {cuda})" if cuda else ")"))
        self.code = code


# ---------------------------------------------------------------------------------------------
# sampler object
# ---------------------------------------------------------------------------------------------

class Sampler:
    """One libsds context with its device buffers.

    Methods mirror the C entry points: reset, draft, verify_window, advance, sample_all,
    sample_all_host, get, set_state, denoise.
    """

    def __init__(self, a, c, sigma, B: int, d: int, L: int, *, gmm_means=None, gmm_logw=None, tcond=None,
                 gmm_bf16: bool = False, mlp=None, callback=None, phi4=None, seed: int = 0, chain_id_offset: int = 0,
                 drafter_mode: int = 0, drafter=None, picard=None, device="cuda:0", stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("libsds needs a CUDA device; there is no CPU path")
        self.torch = torch
        self.lib = load()
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.B, self.d, self.L, self.K = int(B), int(d), int(L), len(a)
        self._keep = []
        a = np.ascontiguousarray(a, np.float32)
        c = np.ascontiguousarray(c, np.float32)
        sigma = np.ascontiguousarray(sigma, np.float32)
        sch = SdsSchedule()
        sch.K = self.K
        sch.a, sch.c, sch.sigma = a.ctypes.data, c.ctypes.data, sigma.ctypes.data
        if tcond is not None:
            tcond = np.ascontiguousarray(tcond, np.float64)
            sch.tcond, sch.tcond_dim = tcond.ctypes.data, tcond.shape[1]
        self._keep += [a, c, sigma, tcond]
        den = self._make_denoiser("tgt", gmm_means, gmm_logw, gmm_bf16, mlp, phi4, callback)
        if den is None:
            raise ValueError("a denoiser is required")
        dden, dtc = None, None
        if drafter is not None:                  # independent draft model: dict(gmm_means=, gmm_logw=, tcond=, gmm_bf16=, mlp=, phi4=)
            dden = self._make_denoiser("drf", drafter.get("gmm_means"), drafter.get("gmm_logw"),
                                       drafter.get("gmm_bf16", False), drafter.get("mlp"), drafter.get("phi4"), None)
            if dden is None:
                raise ValueError("the drafter needs a denoiser")
            if drafter.get("tcond") is not None:
                dtc = np.ascontiguousarray(drafter["tcond"], np.float64)
            drafter_mode = SDS_INDEPENDENT
        self._sch, self._den, self._dden, self._dtc = sch, den, dden, dtc
        nbytes = C.c_size_t(0)
        h = C.c_void_p()
        if picard is not None:                   # (calls, a_det, c_det): Picard drafter
            if dden is not None:
                raise ValueError("picard and drafter exclude each other")
            calls, a_det, c_det = picard
            a_det = np.ascontiguousarray(a_det, np.float32)
            c_det = np.ascontiguousarray(c_det, np.float32)
            if a_det.shape != (self.K,) or c_det.shape != (self.K,):
                raise ValueError("a_det and c_det must have one entry per transition")
            drafter_mode = SDS_PICARD
            self._chk(self.lib.sds_workspace_bytes_picard(C.byref(sch), C.byref(den), self.B, self.d, self.L,
                                                          C.byref(nbytes)), "sds_workspace_bytes_picard")
            self._chk(self.lib.sds_create_picard(C.byref(sch), C.byref(den), int(calls), a_det.ctypes.data,
                                                 c_det.ctypes.data, self.B, self.d, self.L, C.byref(h)),
                      "sds_create_picard")
        elif dden is None:
            self._chk(self.lib.sds_workspace_bytes(C.byref(sch), C.byref(den), self.B, self.d, self.L, C.byref(nbytes)),
                      "sds_workspace_bytes")
            self._chk(self.lib.sds_create(C.byref(sch), C.byref(den), self.B, self.d, self.L, C.byref(h)), "sds_create")
        else:
            tcp = dtc.ctypes.data if dtc is not None else None
            self._chk(self.lib.sds_workspace_bytes_with_drafter(C.byref(sch), C.byref(den), C.byref(dden), tcp, self.B,
                                                                self.d, self.L, C.byref(nbytes)),
                      "sds_workspace_bytes_with_drafter")
            self._chk(self.lib.sds_create_with_drafter(C.byref(sch), C.byref(den), C.byref(dden), tcp, self.B, self.d,
                                                       self.L, C.byref(h)), "sds_create_with_drafter")
        self.h = h
        self.workspace_bytes = nbytes.value
        self.ws = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        base = (self.ws.data_ptr() + 255) // 256 * 256
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._chk(self.lib.sds_bind(self.h, base, nbytes.value, self.stream.cuda_stream, seed, drafter_mode,
                                    chain_id_offset), "sds_bind")

    def _make_denoiser(self, tag, gmm_means, gmm_logw, gmm_bf16, mlp, phi4, callback):
        """Fills an SdsDenoiser and keeps the device arrays it names alive under self.<tag>_*."""
        torch = self.torch
        den = SdsDenoiser()
        if gmm_means is not None:
            means = np.ascontiguousarray(gmm_means, np.float32)
            if gmm_bf16:
                bits = means.view(np.uint32)
                if np.any(bits & np.uint32(0xFFFF)):
                    raise ValueError("gmm_bf16 needs bf16-representable means")
                means_t = torch.from_numpy((bits >> np.uint32(16)).astype(np.uint16).view(np.int16)).to(self.device)
            else:
                means_t = torch.from_numpy(means).to(self.device)
            logw_t = torch.from_numpy(np.ascontiguousarray(gmm_logw, np.float32)).to(self.device)
            setattr(self, tag + "_means", means_t)
            setattr(self, tag + "_logw", logw_t)
            if tag == "tgt":
                self.means, self.logw = means_t, logw_t
            den.kind, den.ncomp = SDS_DEN_GMM, means.shape[0]
            den.means_dev, den.logw_dev = means_t.data_ptr(), logw_t.data_ptr()
            den.means_dtype = SDS_BF16 if gmm_bf16 else SDS_F32
        elif mlp is not None:
            nl = len(mlp.weights)
            dev_bits = lambda x: torch.from_numpy(np.ascontiguousarray(x, np.uint16).view(np.int16)).to(self.device)
            W = [dev_bits(w) for w in mlp.weights]
            bias = [torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(self.device) for x in mlp.bias]
            temb = [dev_bits(x) if x is not None else None for x in mlp.temb]
            dims = np.ascontiguousarray(mlp.dims, np.int32)
            Wp = (C.c_void_p * nl)(*[x.data_ptr() for x in W])
            bp = (C.c_void_p * nl)(*[x.data_ptr() for x in bias])
            tp = (C.c_void_p * nl)(*[(x.data_ptr() if x is not None else None) for x in temb])
            setattr(self, tag + "_mlp", (W, bias, temb, dims, Wp, bp, tp))
            den.kind, den.nlayer = SDS_DEN_MLP, nl
            den.W_dev = C.cast(Wp, C.c_void_p)
            den.bias_dev = C.cast(bp, C.c_void_p)
            den.temb_dev = C.cast(tp, C.c_void_p)
            den.dims = dims.ctypes.data
        elif phi4 is not None:                   # (grid side, coupling beta, periodic)
            den.kind, den.grid_side, den.coupling, den.periodic = SDS_DEN_PHI4, int(phi4[0]), float(phi4[1]), int(bool(phi4[2]))
        elif callback is not None:
            self._cb = DENOISE_FN(callback)
            den.kind, den.fn = SDS_DEN_CALLBACK, self._cb
        else:
            return None
        return den

    # -- helpers --
    def _chk(self, rc: int, where: str, allow=()):
        if rc != SDS_OK and rc not in allow:
            cuda = self.lib.sds_last_cuda_error(self.h) if getattr(self, "h", None) else 0
            raise SdsError(rc, where, cuda)
        return rc

    def close(self):
        if getattr(self, "h", None):
            self.lib.sds_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the path --
    def reset(self):
        self._chk(self.lib.sds_reset(self.h), "sds_reset")

    def draft(self):
        self._chk(self.lib.sds_draft(self.h), "sds_draft")

    def verify_window(self):
        self._chk(self.lib.sds_verify_window(self.h), "sds_verify_window")

    def advance(self, sync: bool = True) -> Optional[int]:
        if not sync:
            self._chk(self.lib.sds_advance(self.h, None), "sds_advance")
            return None
        n = C.c_int64(0)
        self._chk(self.lib.sds_advance(self.h, C.byref(n)), "sds_advance", allow=(SDS_ENONFINITE,))
        return n.value

    def sample_all(self, out=None, nfe_calls=None, nfe_rows=None):
        t = self.torch
        out = out if out is not None else t.empty((self.B, self.d), dtype=t.float32, device=self.device)
        nfe_calls = nfe_calls if nfe_calls is not None else t.empty((self.B,), dtype=t.int32, device=self.device)
        nfe_rows = nfe_rows if nfe_rows is not None else t.empty((self.B,), dtype=t.int32, device=self.device)
        self._chk(self.lib.sds_sample_all(self.h, out.data_ptr(), nfe_calls.data_ptr(), nfe_rows.data_ptr()),
                  "sds_sample_all", allow=(SDS_ENONFINITE,))
        return out, nfe_calls, nfe_rows

    def sample_all_host(self, means_host, logw_host, out_host, nfe_calls_host, nfe_rows_host):
        """Host (pinned) tensors in and out; parameter upload and result download are part of the call."""
        p = lambda x: x.data_ptr() if x is not None else None
        self._chk(self.lib.sds_sample_all_host(self.h, p(means_host), p(logw_host), p(out_host), p(nfe_calls_host),
                                               p(nfe_rows_host)), "sds_sample_all_host", allow=(SDS_ENONFINITE,))

    _GET = {
        GET_X: ("float32", "rows_d"), GET_TAIL: ("float32", "B_d"), GET_DQ: ("float32", "rows_d"),
        GET_DC: ("float32", "B_d"), GET_Y: ("float32", "B_d"), GET_N: ("int32", "B"), GET_ACT: ("int32", "B"),
        GET_ROWOFF: ("int32", "B1"), GET_S1: ("float64", "B_L"), GET_S2: ("float64", "B_L"),
        GET_ELL: ("float32", "B_L"), GET_LOGU: ("float32", "B_L"), GET_ACCMASK: ("uint32", "B"),
        GET_JSTAR: ("int32", "B"), GET_NFE_CALLS: ("int32", "B"), GET_NFE_ROWS: ("int32", "B"),
        GET_CTL: ("int32", "ctl"), GET_ROWK: ("int32", "rows"), GET_DP: ("float32", "rows_d"),
    }

    def get(self, what: int) -> np.ndarray:
        """Host copy of an internal array."""
        dt, shp = self._GET[what]
        B, L, d = self.B, self.L, self.d
        shape = {"rows_d": (B * L, d), "B_d": (B, d), "B": (B,), "B1": (B + 1,), "B_L": (B, L), "ctl": (16,),
                 "rows": (B * L,)}[shp]
        arr = np.empty(shape, dtype=dt)
        self._chk(self.lib.sds_get(self.h, what, arr.ctypes.data, arr.nbytes, 1), "sds_get")
        return arr

    def set_state(self, Y=None, n=None, Dc=None):
        p = lambda x: x.data_ptr() if x is not None else None
        self._keep_state = (Y, n, Dc)
        self._chk(self.lib.sds_set_state(self.h, p(Y), p(n), p(Dc)), "sds_set_state")

    def denoise(self, x, k, out=None):
        t = self.torch
        out = out if out is not None else t.empty_like(x)
        self._chk(self.lib.sds_denoise(self.h, x.data_ptr(), k.data_ptr(), x.shape[0], out.data_ptr()), "sds_denoise")
        return out

    OPT_WHOLE_CHAIN_KERNEL = 1
    OPT_TENSOR_SPLIT = 2
    OPT_GEMM_PAIR = 3
    OPT_VERIFY_EARLY_EXIT = 4
    OPT_FUSE_ADVANCE = 5
    OPT_RAW_ROWS = 6
    OPT_REGEN_DRAFTS = 7
    OPT_ONEHOT_ROWS = 8
    OPT_STAGED_WINDOWS = 9
    STAGED_ADAPTIVE = 255

    def set_option(self, option: int, value: int):
        self._chk(self.lib.sds_set_option(self.h, option, value), "sds_set_option")

    def set_temperature(self, tau: float):
        self._chk(self.lib.sds_set_temperature(self.h, float(tau)), "sds_set_temperature")

    def set_projection(self, Q):
        """Q: float32 CUDA tensor [r, d] with orthonormal rows (see schedules.projection_basis), or None to
        return to the full-space accept test. The tensor is kept alive by this object."""
        if Q is None:
            self._chk(self.lib.sds_set_projection(self.h, None, 0), "sds_set_projection")
            self._proj = None
            return
        t = self.torch
        if Q.dtype != t.float32 or not Q.is_cuda or Q.dim() != 2 or Q.shape[1] != self.d or not Q.is_contiguous():
            raise ValueError("Q must be a contiguous float32 CUDA tensor [r, d]")
        self._chk(self.lib.sds_set_projection(self.h, Q.data_ptr(), int(Q.shape[0])), "sds_set_projection")
        self._proj = Q

    PROF_KINDS = ("init", "denoise", "draft", "verify", "advance", "fused", "aux", "softmax", "draft_model", "mix")

    def profile(self, enable: bool):
        self._chk(self.lib.sds_profile(self.h, int(enable)), "sds_profile")

    def profile_read(self, reset: bool = True) -> dict:
        """{kind: (milliseconds, launches)} accumulated since the last reset."""
        ms = np.zeros(len(self.PROF_KINDS), np.float64)
        n = np.zeros(len(self.PROF_KINDS), np.int64)
        self._chk(self.lib.sds_profile_read(self.h, ms.ctypes.data, n.ctypes.data, int(reset)), "sds_profile_read")
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(self.PROF_KINDS)}

    def launch_count(self) -> int:
        return int(self.lib.sds_launch_count(self.h))


def rng_normals(seed: int, stream_id: int, b0: int, nb: int, k: int, d: int, device="cuda:0"):
    import torch
    out = torch.empty((nb, d), dtype=torch.float32, device=device)
    rc = load().sds_rng_normals(seed, stream_id, b0, nb, k, d, out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    if rc != SDS_OK:
        raise SdsError(rc, "sds_rng_normals")
    return out


def rng_uniforms(seed: int, b0: int, nb: int, k: int, device="cuda:0"):
    import torch
    out = torch.empty((nb,), dtype=torch.float32, device=device)
    rc = load().sds_rng_uniforms(seed, b0, nb, k, out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    if rc != SDS_OK:
        raise SdsError(rc, "sds_rng_uniforms")
    return out


STATIC_MAX_NCOMP = 4096


def gmm_denoise_static(x, k, means, logw, tcond, out):
    """sds_gmm_denoise_static on torch CUDA tensors (all caller-allocated, including out): a mixture
    denoiser pass for callers that cannot allocate device memory. Enqueues on the current stream."""
    import torch
    rc = load().sds_gmm_denoise_static(x.data_ptr(), k.data_ptr(), x.shape[0], x.shape[1], means.shape[0],
                                       means.data_ptr(), logw.data_ptr(), tcond.data_ptr(), tcond.shape[0],
                                       out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    if rc != SDS_OK:
        raise SdsError(rc, "sds_gmm_denoise_static")
    return out
