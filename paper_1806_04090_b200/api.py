"""Thin Python binding of the C ABI in ``include/atomo.h`` (argument marshalling only).

Every step of the encode / decode path runs in the CUDA library; PyTorch is used for device
memory and streams.  There is no CPU fallback: if the shared library is missing or no CUDA
device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ATOMO_B200_LIB", os.path.join(_HERE, "libatomo_b200.so"))

KIND_SPECTRAL = 0
KIND_ENTRYWISE = 1
EW_EXPLICIT, EW_COMPACT = 0, 1      # entry-wise payload formats
EW_TILE = 4096                       # elements per tile of the entry-wise offset table
STATUS_NAMES = ["OK", "INVALID_ARG", "BUDGET", "CAPACITY", "NONFINITE", "NOT_CONVERGED", "TIMEOUT", "CUDA",
                "PAYLOAD"]
STAGES = ["gram", "eig", "sample", "backproject", "ew_reduce", "ew_pack", "decode"]

# every symbol include/atomo.h declares
EXPORTS = [
    "atomo_create", "atomo_destroy", "atomo_last_cuda_error", "atomo_payload_bytes_spectral",
    "atomo_payload_bytes_entrywise", "atomo_encode_spectral", "atomo_encode_entrywise", "atomo_decode",
    "atomo_payload_read_headers", "atomo_payload_status", "atomo_set_profiling", "atomo_get_stage_times",
    "atomo_set_eig_params", "atomo_set_eig_mode", "atomo_set_sigma_refinement", "atomo_set_gram_path", "atomo_set_persistent_eig", "atomo_last_eig_scheme", "atomo_decode_spectral_static", "atomo_decode_average", "atomo_lq_budget",
    "atomo_payload_bytes_entrywise_compact", "atomo_set_entrywise_format", "atomo_get_stage_totals",
    "atomo_set_tridiag_ctas", "atomo_measure_fma_peak", "atomo_encode_spectral_from_svd", "atomo_get_table_uploads",
    "atomo_set_entrywise_launch",
    "atomo_get_entrywise_list_chunks",
]


class AtomoError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{where}: ATOMO_ERR_{name}" + (f" ({detail})" if detail else ""))
        self.code = code


class _Mat(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("rows", ctypes.c_int32), ("cols", ctypes.c_int32), ("ld", ctypes.c_int64)]


class _Vec(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("n", ctypes.c_int64)]


class _Debug(ctypes.Structure):
    _fields_ = [("sigma", ctypes.c_void_p), ("prob", ctypes.c_void_p), ("mask_words", ctypes.c_void_p),
                ("short_vecs", ctypes.c_void_p)]


class PayloadHeader(ctypes.Structure):
    _fields_ = [("magic", ctypes.c_uint32), ("version", ctypes.c_uint32), ("kind", ctypes.c_uint32),
                ("n_layers", ctypes.c_uint32), ("total_bytes", ctypes.c_uint64), ("seed", ctypes.c_uint64),
                ("step", ctypes.c_uint64), ("s", ctypes.c_double), ("ew_format", ctypes.c_uint64), ("ew_sat_cap", ctypes.c_uint64)]


class LayerHeader(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("k_cap", ctypes.c_uint32), ("k", ctypes.c_uint32),
                ("n_sat", ctypes.c_uint32), ("status", ctypes.c_uint32), ("c", ctypes.c_float),
                ("sweeps", ctypes.c_uint32), ("off_idx", ctypes.c_uint64), ("off_val", ctypes.c_uint64),
                ("off_short", ctypes.c_uint64), ("off_long", ctypes.c_uint64), ("l1", ctypes.c_double)]


assert ctypes.sizeof(PayloadHeader) == 64 and ctypes.sizeof(LayerHeader) == 80

_lib = None


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    """Load libatomo_b200.so (no CUDA call is made by loading)."""
    global _lib
    if _lib is not None and path == LIB_PATH:
        return _lib
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_1806_04090_b200.build` (there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, i32, i64, u64, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
    lib.atomo_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
    lib.atomo_destroy.argtypes = [vp]
    lib.atomo_last_cuda_error.argtypes = [vp]
    lib.atomo_last_cuda_error.restype = ctypes.c_char_p
    lib.atomo_payload_bytes_spectral.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32), i32, i32]
    lib.atomo_payload_bytes_spectral.restype = i64
    lib.atomo_payload_bytes_entrywise.argtypes = [ctypes.POINTER(i64), i32, i64]
    lib.atomo_payload_bytes_entrywise.restype = i64
    lib.atomo_payload_bytes_entrywise_compact.argtypes = [ctypes.POINTER(i64), i32, i64, i64]
    lib.atomo_payload_bytes_entrywise_compact.restype = i64
    lib.atomo_set_entrywise_format.argtypes = [vp, i32, i64]
    lib.atomo_set_entrywise_launch.argtypes = [vp, i32]
    lib.atomo_get_entrywise_list_chunks.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint32)]
    lib.atomo_encode_spectral.argtypes = [vp, ctypes.POINTER(_Mat), i32, dbl, u64, u64, i32, vp, i64,
                                          ctypes.POINTER(_Debug), vp]
    lib.atomo_encode_entrywise.argtypes = [vp, ctypes.POINTER(_Vec), i32, dbl, u64, u64, i64, vp, i64,
                                           ctypes.POINTER(_Debug), vp]
    lib.atomo_decode.argtypes = [vp, i32, vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(vp), i32, vp]
    lib.atomo_decode_average.argtypes = [vp, i32, ctypes.POINTER(vp), i32, ctypes.POINTER(i64), ctypes.POINTER(i64),
                                         ctypes.POINTER(vp), i32, vp]
    lib.atomo_lq_budget.argtypes = [vp, ctypes.POINTER(_Vec), i32, dbl, ctypes.POINTER(dbl), vp]
    lib.atomo_payload_read_headers.argtypes = [vp, vp, i32, ctypes.POINTER(PayloadHeader),
                                               ctypes.POINTER(LayerHeader), vp]
    lib.atomo_payload_status.argtypes = [vp, vp, i32, ctypes.POINTER(i32), ctypes.POINTER(i32), vp]
    lib.atomo_set_profiling.argtypes = [vp, ctypes.c_int]
    lib.atomo_get_stage_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i64)]
    lib.atomo_get_stage_totals.argtypes = [vp, ctypes.POINTER(dbl), ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.atomo_set_eig_params.argtypes = [vp, i32, ctypes.c_float]
    lib.atomo_set_eig_mode.argtypes = [vp, i32]
    lib.atomo_set_sigma_refinement.argtypes = [vp, i32]
    lib.atomo_set_gram_path.argtypes = [vp, i32]
    lib.atomo_set_persistent_eig.argtypes = [vp, i32]
    lib.atomo_last_eig_scheme.argtypes = [vp]
    lib.atomo_set_tridiag_ctas.argtypes = [vp, i32]
    lib.atomo_get_table_uploads.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.atomo_encode_spectral_from_svd.argtypes = [vp, ctypes.POINTER(_Mat), i32, ctypes.POINTER(vp), ctypes.POINTER(vp),
                                                   ctypes.c_double, u64, u64, i32, vp, i64, ctypes.POINTER(_Debug), vp]
    lib.atomo_measure_fma_peak.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_double)]
    lib.atomo_decode_spectral_static.argtypes = [ctypes.c_int, vp, ctypes.POINTER(i64), ctypes.POINTER(i64),
                                                 ctypes.POINTER(vp), i32, vp]
    if path == LIB_PATH:
        _lib = lib
    return lib


def payload_bytes_spectral(shapes: Sequence[Sequence[int]], k_cap: int) -> int:
    lib = load_library()
    n = len(shapes)
    rows = (ctypes.c_int32 * n)(*[int(s[0]) for s in shapes])
    cols = (ctypes.c_int32 * n)(*[int(s[1]) for s in shapes])
    return int(lib.atomo_payload_bytes_spectral(rows, cols, n, int(k_cap)))


def payload_bytes_entrywise(lengths: Sequence[int], k_cap: int) -> int:
    lib = load_library()
    n = len(lengths)
    arr = (ctypes.c_int64 * n)(*[int(x) for x in lengths])
    return int(lib.atomo_payload_bytes_entrywise(arr, n, int(k_cap)))


def payload_bytes_entrywise_compact(lengths: Sequence[int], k_cap: int, sat_cap: int) -> int:
    lib = load_library()
    n = len(lengths)
    arr = (ctypes.c_int64 * n)(*[int(x) for x in lengths])
    return int(lib.atomo_payload_bytes_entrywise_compact(arr, n, int(k_cap), int(sat_cap)))


def measure_fma_peak(device: int = 0, fp64: bool = False) -> float:
    """Measured FMA rate of the GPU in TFLOP/s (fp32 or fp64), see atomo_measure_fma_peak."""
    out = ctypes.c_double(0.0)
    rc = load_library().atomo_measure_fma_peak(int(device), 1 if fp64 else 0, ctypes.byref(out))
    if rc != 0:
        raise AtomoError(rc, "atomo_measure_fma_peak")
    return float(out.value)


def default_k_cap(s: float, n_atoms: int) -> int:
    """k is a sum of independent Bernoulli draws with mean <= s: s + 8 sqrt(s) + 8 is never reached."""
    return int(min(n_atoms, np.ceil(s + 8.0 * np.sqrt(max(float(s), 0.0)) + 8.0)))


@dataclass
class Debug:
    """Optional per-atom outputs (device tensors) for parity checks."""
    sigma: Optional[torch.Tensor] = None
    prob: Optional[torch.Tensor] = None
    mask_words: Optional[torch.Tensor] = None
    short_vecs: Optional[torch.Tensor] = None
    atom_offsets: List[int] = field(default_factory=list)
    word_offsets: List[int] = field(default_factory=list)
    sq_offsets: List[int] = field(default_factory=list)

    def layer_mask(self, l: int, n_atoms: int) -> np.ndarray:
        w0 = self.word_offsets[l]
        words = self.mask_words[w0: w0 + (n_atoms + 31) // 32].cpu().numpy().astype(np.uint32)
        bits = np.unpackbits(words.view(np.uint8), bitorder="little")
        return bits[:n_atoms].astype(bool)

    def layer_prob(self, l: int, n_atoms: int) -> np.ndarray:
        a0 = self.atom_offsets[l]
        return self.prob[a0: a0 + n_atoms].cpu().numpy()

    def layer_sigma(self, l: int, n_atoms: int) -> np.ndarray:
        a0 = self.atom_offsets[l]
        return self.sigma[a0: a0 + n_atoms].cpu().numpy()

    def layer_short(self, l: int, r: int) -> np.ndarray:
        o = self.sq_offsets[l]
        return self.short_vecs[o: o + r * r].cpu().numpy().reshape(r, r)


@dataclass
class Payload:
    """A device payload plus the host-side facts needed to decode it."""
    buf: torch.Tensor            # uint8, device
    kind: int
    shapes: List[tuple]          # (rows, cols) per layer; entry-wise: (1, n)
    k_cap: int
    ctx: "Atomo"
    ew_format: int = 0           # entry-wise: EW_EXPLICIT or EW_COMPACT
    sat_cap: int = 0             # compact entry-wise: capacity of the saturated list

    @property
    def n_layers(self) -> int:
        return len(self.shapes)

    def headers(self):
        return self.ctx.read_headers(self)

    def layer_arrays(self, l: int, hdrs=None):
        """Host copies of one layer's kept atoms (test / inspection helper)."""
        _, lh = hdrs if hdrs is not None else self.headers()
        h = lh[l]
        k = int(h.k)
        raw = self.buf

        def view(off, count, dtype):
            nbytes = count * 4
            return raw[off: off + nbytes].cpu().numpy().view(dtype)

        if self.kind == KIND_ENTRYWISE and self.ew_format == EW_COMPACT:
            # expand the compact form to the explicit (idx, val) pair: entries carry the index inside their tile
            # and the sign of +-c; the saturated atoms sit in a list of their own
            n = self.shapes[l][1]
            n_sat = int(h.n_sat)
            k_list = k - n_sat
            n_tiles = (n + EW_TILE - 1) // EW_TILE
            ent = raw[h.off_idx: h.off_idx + 2 * k_list].cpu().numpy().view(np.uint16).astype(np.int64)
            table = view(h.off_short, n_tiles + 1, np.uint32).astype(np.int64)
            tile_of = np.searchsorted(table[1:], np.arange(k_list), side="right")
            idx_u = tile_of * EW_TILE + (ent & (EW_TILE - 1))
            val_u = np.where(ent & 0x8000, -np.float32(h.c), np.float32(h.c)).astype(np.float32)
            idx_s = view(h.off_long, n_sat, np.uint32).astype(np.int64)
            val_s = view(h.off_val, n_sat, np.float32)
            idx = np.concatenate([idx_u, idx_s])
            val = np.concatenate([val_u, val_s])
            order = np.argsort(idx, kind="stable")
            return dict(k=k, idx=idx[order].astype(np.uint32), val=val[order].astype(np.float32),
                        n_sat_kept=n_sat, table=table)
        idx = view(h.off_idx, k, np.uint32).copy()
        val = view(h.off_val, k, np.float32).copy()
        if self.kind == KIND_ENTRYWISE:
            return dict(k=k, idx=idx, val=val)
        rows, cols = self.shapes[l]
        r, L = min(rows, cols), max(rows, cols)
        short = view(h.off_short, k * r, np.float32).reshape(k, r).copy()
        long_ = view(h.off_long, k * L, np.float32).reshape(k, L).copy()
        U, V = (short, long_) if rows <= cols else (long_, short)
        return dict(k=k, idx=idx, coef=val, U=U.T.copy(), V=V.T.copy())


def atomo_decode_spectral_static(payload: "Payload", out: Sequence[torch.Tensor], device: Optional[int] = None,
                                 stream: Optional[torch.cuda.Stream] = None) -> List[torch.Tensor]:
    """Spectral decode that allocates nothing on the device: for processes whose framework
    allocator owns the whole GPU, or that cannot take cudaMalloc's device-wide synchronisation
    where they decode.  The caller supplies the output tensors; the per-call tables live in a fixed
    array inside the library (limits: 64 layers, 8192 output tiles of 64 x 1024).  Calls on one
    device share that array, so they must not overlap on the GPU.  Every output must be a contiguous
    fp32 CUDA tensor on the payload's device with exactly rows * cols elements: the kernel writes all
    of them through the raw pointer, so anything else is refused here, before the C call."""
    lib = load_library()
    if payload.kind != KIND_SPECTRAL:
        raise ValueError("atomo_decode_spectral_static decodes spectral payloads only")
    n = payload.n_layers
    if len(out) != n:
        raise ValueError("one output tensor per layer is required (this call does not allocate)")
    dev = payload.buf.device.index if device is None else int(device)
    for l, (o, (r_, c_)) in enumerate(zip(out, payload.shapes)):
        if not (isinstance(o, torch.Tensor) and o.is_cuda and o.device.index == dev and o.dtype == torch.float32
                and o.is_contiguous() and o.numel() == int(r_) * int(c_)):
            raise ValueError(f"output {l}: a contiguous fp32 CUDA tensor on device {dev} with {int(r_) * int(c_)} elements is required")
    rows = (ctypes.c_int64 * n)(*[r for r, _ in payload.shapes])
    cols = (ctypes.c_int64 * n)(*[c for _, c in payload.shapes])
    ptrs = (ctypes.c_void_p * n)(*[o.data_ptr() for o in out])
    s = stream if stream is not None else torch.cuda.current_stream()
    rc = lib.atomo_decode_spectral_static(dev, ctypes.c_void_p(payload.buf.data_ptr()), rows, cols, ptrs, n,
                                          ctypes.c_void_p(s.cuda_stream))
    if rc != 0:
        raise AtomoError(rc, "atomo_decode_spectral_static",
                         "batch exceeds the fixed table (64 layers / 8192 tiles)" if rc == 3 else "")
    return list(out)


class Atomo:
    """One library context bound to a CUDA device."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("atomo: no CUDA device available (the library has no CPU fallback)")
        self.lib = load_library()
        self.device = int(device)
        torch.cuda.init()
        h = ctypes.c_void_p()
        rc = self.lib.atomo_create(ctypes.byref(h), self.device)
        self._h = h
        self._ew_format, self._ew_sat_cap = EW_EXPLICIT, 0
        if rc != 0:
            raise AtomoError(rc, "atomo_create", self._cuda_error())

    def _cuda_error(self) -> str:
        try:
            return (self.lib.atomo_last_cuda_error(self._h) or b"").decode()
        except Exception:  # pragma: no cover
            return ""

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.atomo_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != 0:
            raise AtomoError(rc, where, self._cuda_error() if rc == 7 else "")

    @staticmethod
    def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
        s = stream if stream is not None else torch.cuda.current_stream()
        return ctypes.c_void_p(s.cuda_stream)

    def _make_debug(self, n_atoms: Sequence[int], spectral: bool, want_short: bool, dev, want_prob: bool = True) -> Debug:
        a_off = np.concatenate([[0], np.cumsum(n_atoms)]).astype(np.int64)
        w_off = np.concatenate([[0], np.cumsum([(n + 31) // 32 for n in n_atoms])]).astype(np.int64)
        sq_off = np.concatenate([[0], np.cumsum([n * n for n in n_atoms])]).astype(np.int64)
        d = Debug(atom_offsets=a_off.tolist(), word_offsets=w_off.tolist(), sq_offsets=sq_off.tolist())
        if want_prob:
            d.prob = torch.zeros(int(a_off[-1]), dtype=torch.float32, device=dev)
        d.mask_words = torch.zeros(int(w_off[-1]), dtype=torch.int32, device=dev)
        if spectral:
            d.sigma = torch.zeros(int(a_off[-1]), dtype=torch.float32, device=dev)
            if want_short:
                d.short_vecs = torch.zeros(int(sq_off[-1]), dtype=torch.float32, device=dev)
        return d

    @staticmethod
    def _debug_struct(d: Optional[Debug]):
        if d is None:
            return None
        ptr = lambda t: ctypes.c_void_p(t.data_ptr()) if t is not None else None
        return _Debug(ptr(d.sigma), ptr(d.prob), ptr(d.mask_words), ptr(d.short_vecs))

    # ------------------------------------------------------------------------------------------
    def atomo_encode_spectral(self, layers: Sequence[torch.Tensor], s: float, seed: int, step: int = 0,
                              k_cap: Optional[int] = None, payload: Optional[torch.Tensor] = None,
                              debug: bool = False, debug_short: bool = False,
                              stream: Optional[torch.cuda.Stream] = None):
        """Spectral ATOMO over a batch of 2-D fp32 CUDA tensors.  Returns (Payload, Debug | None)."""
        n = len(layers)
        mats = (_Mat * n)()
        shapes = []
        for i, g in enumerate(layers):
            if not (g.is_cuda and g.dtype == torch.float32 and g.dim() == 2 and g.stride(1) == 1):
                raise ValueError("layers must be 2-D fp32 CUDA tensors with unit column stride")
            mats[i] = _Mat(g.data_ptr(), g.shape[0], g.shape[1], g.stride(0) if g.shape[0] > 1 else g.shape[1])
            shapes.append((int(g.shape[0]), int(g.shape[1])))
        if k_cap is None:
            k_cap = default_k_cap(s, max(min(r, c) for r, c in shapes))
        nbytes = payload_bytes_spectral(shapes, k_cap)
        if nbytes < 0:
            raise AtomoError(1, "atomo_payload_bytes_spectral")
        dev = layers[0].device
        if payload is None:
            payload = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        dbg = self._make_debug([min(r, c) for r, c in shapes], True, debug_short, dev) if (debug or debug_short) else None
        ds = self._debug_struct(dbg)
        rc = self.lib.atomo_encode_spectral(self._h, mats, n, float(s), int(seed), int(step), int(k_cap),
                                            ctypes.c_void_p(payload.data_ptr()), payload.numel(),
                                            ctypes.byref(ds) if ds is not None else None, self._stream_ptr(stream))
        self._check(rc, "atomo_encode_spectral")
        return Payload(payload, KIND_SPECTRAL, shapes, int(k_cap), self), dbg

    def atomo_encode_spectral_from_svd(self, layers: Sequence[torch.Tensor], sigma: Sequence[torch.Tensor],
                                       short_vecs: Sequence[torch.Tensor], s: float, seed: int, step: int = 0,
                                       k_cap: Optional[int] = None, debug: bool = True,
                                       stream: Optional[torch.cuda.Stream] = None):
        """Test entry point: the path downstream of the SVD for a decomposition given by the caller.  sigma[l]: r
        fp32 values, descending; short_vecs[l]: r x r fp32, row i = the unit short-side vector of atom i."""
        n = len(layers)
        mats = (_Mat * n)()
        shapes = []
        for i, g in enumerate(layers):
            if not (g.is_cuda and g.dtype == torch.float32 and g.dim() == 2 and g.is_contiguous()):
                raise ValueError("layers must be contiguous 2-D fp32 CUDA tensors")
            r = min(g.shape)
            for t, want in ((sigma[i], r), (short_vecs[i], r * r)):
                if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() == want):
                    raise ValueError("sigma / short_vecs must be contiguous fp32 CUDA tensors of r and r * r elements")
            mats[i] = _Mat(g.data_ptr(), g.shape[0], g.shape[1], g.shape[1])
            shapes.append((int(g.shape[0]), int(g.shape[1])))
        if k_cap is None:
            k_cap = default_k_cap(s, max(min(r, c) for r, c in shapes))
        payload = torch.empty(payload_bytes_spectral(shapes, k_cap), dtype=torch.uint8, device=layers[0].device)
        dbg = self._make_debug([min(r, c) for r, c in shapes], True, False, layers[0].device) if debug else None
        ds = self._debug_struct(dbg)
        sp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in sigma])
        vp_ = (ctypes.c_void_p * n)(*[t.data_ptr() for t in short_vecs])
        rc = self.lib.atomo_encode_spectral_from_svd(self._h, mats, n, sp, vp_, float(s), int(seed), int(step), int(k_cap),
                                                     ctypes.c_void_p(payload.data_ptr()), payload.numel(),
                                                     ctypes.byref(ds) if ds is not None else None, self._stream_ptr(stream))
        self._check(rc, "atomo_encode_spectral_from_svd")
        return Payload(payload, KIND_SPECTRAL, shapes, int(k_cap), self), dbg

    def atomo_encode_entrywise(self, vecs: Sequence[torch.Tensor], s: float, seed: int, step: int = 0,
                               k_cap: Optional[int] = None, payload: Optional[torch.Tensor] = None,
                               debug=False, stream: Optional[torch.cuda.Stream] = None):
        """Entry-wise ATOMO over a batch of flat fp32 CUDA tensors.  Returns (Payload, Debug | None).
        The payload format is the one last chosen with set_entrywise_format (explicit by default).
        debug: True = probabilities and mask words, "mask" = the mask words alone (asking for the probabilities makes
        the one-kernel form read every vector twice)."""
        n = len(vecs)
        arr = (_Vec * n)()
        lengths = []
        for i, g in enumerate(vecs):
            if not (g.is_cuda and g.dtype == torch.float32 and g.is_contiguous()):
                raise ValueError("vectors must be contiguous fp32 CUDA tensors")
            arr[i] = _Vec(g.data_ptr(), g.numel())
            lengths.append(int(g.numel()))
        if k_cap is None:
            k_cap = default_k_cap(s, max(lengths))
        if self._ew_format == EW_COMPACT:
            nbytes = payload_bytes_entrywise_compact(lengths, k_cap, self._ew_sat_cap)
        else:
            nbytes = payload_bytes_entrywise(lengths, k_cap)
        if nbytes < 0:
            raise AtomoError(1, "atomo_payload_bytes_entrywise")
        dev = vecs[0].device
        if payload is None:
            payload = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        dbg = self._make_debug(lengths, False, False, dev, want_prob=(debug != "mask")) if debug else None
        ds = self._debug_struct(dbg)
        rc = self.lib.atomo_encode_entrywise(self._h, arr, n, float(s), int(seed), int(step), int(k_cap),
                                             ctypes.c_void_p(payload.data_ptr()), payload.numel(),
                                             ctypes.byref(ds) if ds is not None else None, self._stream_ptr(stream))
        self._check(rc, "atomo_encode_entrywise")
        return Payload(payload, KIND_ENTRYWISE, [(1, x) for x in lengths], int(k_cap), self,
                       ew_format=self._ew_format, sat_cap=self._ew_sat_cap), dbg

    def atomo_decode(self, payload: Payload, out: Optional[Sequence[torch.Tensor]] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> List[torch.Tensor]:
        """Dense fp32 gradients from a payload (one tensor per layer)."""
        n = payload.n_layers
        dev = payload.buf.device
        if out is None:
            out = [torch.empty(r * c, dtype=torch.float32, device=dev).view((c,) if payload.kind == KIND_ENTRYWISE else (r, c))
                   for r, c in payload.shapes]
        rows = (ctypes.c_int64 * n)(*[r for r, _ in payload.shapes])
        cols = (ctypes.c_int64 * n)(*[c for _, c in payload.shapes])
        ptrs = (ctypes.c_void_p * n)(*[o.data_ptr() for o in out])
        rc = self.lib.atomo_decode(self._h, payload.kind, ctypes.c_void_p(payload.buf.data_ptr()), rows, cols, ptrs, n,
                                   self._stream_ptr(stream))
        self._check(rc, "atomo_decode")
        return list(out)

    # ------------------------------------------------------------------------------------------
    def atomo_decode_average(self, payloads: Sequence[Payload], out: Optional[Sequence[torch.Tensor]] = None,
                             stream: Optional[torch.cuda.Stream] = None) -> List[torch.Tensor]:
        """Mean of the dense gradients of several payloads of the same shapes (the workers' payloads after an
        all-gather), one tensor per layer, in one pass over the output."""
        if len(payloads) == 0:
            raise ValueError("atomo_decode_average needs at least one payload")
        first = payloads[0]
        for p in payloads[1:]:
            if p.kind != first.kind or list(p.shapes) != list(first.shapes):
                raise ValueError("payloads of one average must share kind and shapes")
        n = first.n_layers
        dev = first.buf.device
        if out is None:
            out = [torch.empty(r * c, dtype=torch.float32, device=dev).view((c,) if first.kind == KIND_ENTRYWISE else (r, c))
                   for r, c in first.shapes]
        rows = (ctypes.c_int64 * n)(*[r for r, _ in first.shapes])
        cols = (ctypes.c_int64 * n)(*[c for _, c in first.shapes])
        ptrs = (ctypes.c_void_p * n)(*[o.data_ptr() for o in out])
        pays = (ctypes.c_void_p * len(payloads))(*[p.buf.data_ptr() for p in payloads])
        rc = self.lib.atomo_decode_average(self._h, first.kind, pays, len(payloads), rows, cols, ptrs, n,
                                           self._stream_ptr(stream))
        self._check(rc, "atomo_decode_average")
        return list(out)

    def atomo_lq_budget(self, vecs: Sequence[torch.Tensor], q: float, stream: Optional[torch.cuda.Stream] = None) -> List[float]:
        """s = ||g||_1 / ||g||_q per vector (Section 4: q = 2 is QSGD's budget, q = inf TernGrad's)."""
        n = len(vecs)
        arr = (_Vec * n)()
        for i, v in enumerate(vecs):
            if v.dtype != torch.float32 or not v.is_cuda or not v.is_contiguous():
                raise ValueError("vectors must be contiguous fp32 CUDA tensors")
            arr[i].data = v.data_ptr(); arr[i].n = v.numel()
        out = (ctypes.c_double * n)()
        self._check(self.lib.atomo_lq_budget(self._h, arr, n, float(q), out, self._stream_ptr(stream)), "atomo_lq_budget")
        return [float(x) for x in out]

    def read_headers(self, payload: Payload, stream: Optional[torch.cuda.Stream] = None):
        gh = PayloadHeader()
        lh = (LayerHeader * payload.n_layers)()
        rc = self.lib.atomo_payload_read_headers(self._h, ctypes.c_void_p(payload.buf.data_ptr()), payload.n_layers,
                                                 ctypes.byref(gh), lh, self._stream_ptr(stream))
        self._check(rc, "atomo_payload_read_headers")
        return gh, list(lh)

    def payload_status(self, payload: Payload, stream: Optional[torch.cuda.Stream] = None):
        worst, first = ctypes.c_int32(0), ctypes.c_int32(-1)
        rc = self.lib.atomo_payload_status(self._h, ctypes.c_void_p(payload.buf.data_ptr()), payload.n_layers,
                                           ctypes.byref(worst), ctypes.byref(first), self._stream_ptr(stream))
        self._check(rc, "atomo_payload_status")
        return int(worst.value), int(first.value)

    def set_profiling(self, on: bool):
        self._check(self.lib.atomo_set_profiling(self._h, 1 if on else 0), "atomo_set_profiling")

    def stage_times(self):
        ms = (ctypes.c_float * len(STAGES))()
        ln = (ctypes.c_int64 * len(STAGES))()
        self._check(self.lib.atomo_get_stage_times(self._h, ms, ln), "atomo_get_stage_times")
        return {k: float(ms[i]) for i, k in enumerate(STAGES)}, {k: int(ln[i]) for i, k in enumerate(STAGES)}

    def stage_totals(self):
        """(ms per stage, launches per stage, calls) summed over all encode / decode calls since profiling was switched
        on; the calls themselves do not wait for their events, this does."""
        ms = (ctypes.c_double * len(STAGES))()
        ln = (ctypes.c_int64 * len(STAGES))()
        calls = ctypes.c_int64(0)
        self._check(self.lib.atomo_get_stage_totals(self._h, ms, ln, ctypes.byref(calls)), "atomo_get_stage_totals")
        return ({k: float(ms[i]) for i, k in enumerate(STAGES)}, {k: int(ln[i]) for i, k in enumerate(STAGES)},
                int(calls.value))

    def set_persistent_eig(self, enabled):
        """Eigen-solver scheme.  0 / False: Jacobi, one launch per step; 1 / True: persistent cooperative launches;
        2: Jacobi in thread-block clusters first; 3 (default): the tridiagonal routes (any short side up to 4096)."""
        self._check(self.lib.atomo_set_persistent_eig(self._h, int(enabled)), "atomo_set_persistent_eig")

    def set_entrywise_format(self, fmt: int, sat_cap: int = 0):
        """EW_EXPLICIT (idx, val per kept atom) or EW_COMPACT (16-bit entry per kept atom with p < 1, one scalar c,
        explicit values only for the atoms with p = 1, of which at most sat_cap per vector)."""
        self._check(self.lib.atomo_set_entrywise_format(self._h, int(fmt), int(sat_cap)), "atomo_set_entrywise_format")
        self._ew_format, self._ew_sat_cap = int(fmt), (int(sat_cap) if int(fmt) == EW_COMPACT else 0)

    def set_entrywise_launch(self, two_kernels):
        """0 / False (default): one cooperative kernel per vector that fits one wave of resident CTAs, the keep decisions
        taken on the candidate list of its first pass where that holds every kept atom; 1 / True: always the solve kernel
        followed by the sample / pack kernel; 2: the one-kernel form without the list.  Same payloads in every form."""
        self._check(self.lib.atomo_set_entrywise_launch(self._h, int(two_kernels)), "atomo_set_entrywise_launch")

    def entrywise_list_chunks(self, vec: int = 0):
        """(chunks of the last entry-wise encode of vector `vec` that decided on their candidate list, chunks of the
        one-kernel form: 0 if the two-kernel form ran).  Synchronises."""
        a, b = ctypes.c_uint32(0), ctypes.c_uint32(0)
        self._check(self.lib.atomo_get_entrywise_list_chunks(self._h, int(vec), ctypes.byref(a), ctypes.byref(b)),
                    "atomo_get_entrywise_list_chunks")
        return int(a.value), int(b.value)

    def table_uploads(self):
        """(calls that uploaded their descriptor tables, calls that found them on the device) since the context was made."""
        up, re = ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(self.lib.atomo_get_table_uploads(self._h, ctypes.byref(up), ctypes.byref(re)), "atomo_get_table_uploads")
        return int(up.value), int(re.value)

    def set_tridiag_ctas(self, ctas_per_layer: int):
        """CTAs per layer of the blocked tridiagonal reduction (short sides above 512): 0 = chosen per batch, else 1,
        2, 4, 8 or 16.  The payload does not depend on it."""
        self._check(self.lib.atomo_set_tridiag_ctas(self._h, int(ctas_per_layer)), "atomo_set_tridiag_ctas")

    def last_eig_scheme(self) -> int:
        return int(self.lib.atomo_last_eig_scheme(self._h))

    def set_gram_path(self, tensor_cores: bool):
        self._check(self.lib.atomo_set_gram_path(self._h, 1 if tensor_cores else 0), "atomo_set_gram_path")

    def set_sigma_refinement(self, min_short_side: int):
        self._check(self.lib.atomo_set_sigma_refinement(self._h, int(min_short_side)), "atomo_set_sigma_refinement")

    def set_eig_mode(self, mode: int):
        self._check(self.lib.atomo_set_eig_mode(self._h, int(mode)), "atomo_set_eig_mode")

    def set_eig_params(self, max_sweeps: int, tol: float):
        self._check(self.lib.atomo_set_eig_params(self._h, int(max_sweeps), float(tol)), "atomo_set_eig_params")
