"""Thin ctypes binding of liboq.so: same names as the C entry points, argument marshalling only.

Device buffers are torch CUDA tensors (torch owns memory and streams); every step of the path runs in
the library's kernels.  There is no fallback: if liboq.so is missing or a call fails, OqError is raised.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboq.so")
_lib = None

OQ_BF16, OQ_F32 = 0, 1
STATUS_NAMES = {0: "OQ_OK", 1: "OQ_ERR_INVALID_ARG", 2: "OQ_ERR_UNSUPPORTED", 3: "OQ_ERR_ALIGNMENT",
                4: "OQ_ERR_CUDA", 5: "OQ_ERR_DEVICE_TIMEOUT", 6: "OQ_ERR_NOMEM"}


class OqError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {msg}")
        self.code = code


def lib():
    """Loads liboq.so (built in-tree by paper_2607_02461_b200.build); fails loudly when absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise OqError(4, f"{_LIB_PATH} not found: run `python -m paper_2607_02461_b200.build`")
        L = C.CDLL(_LIB_PATH)
        vp, i, u64, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
        pp = C.POINTER(C.c_void_p)
        sig = {
            "oq_build_codebook": (i, [i, i, pp]),
            "oq_codebook_get": (i, [vp, vp, vp, vp, vp]),
            "oq_codebook_dim": (i, [vp]), "oq_codebook_bits": (i, [vp]), "oq_codebook_destroy": (None, [vp]),
            "oq_make_rpbh": (i, [i, i, u64, pp]),
            "oq_rpbh_get": (i, [vp, vp, vp]),
            "oq_rpbh_dim": (i, [vp]), "oq_rpbh_block": (i, [vp]), "oq_rpbh_destroy": (None, [vp]),
            "oq_packed_bytes": (i, [i, i, i, C.POINTER(sz), C.POINTER(sz)]),
            "oq_rotate_quantize_act": (i, [vp, i, i, i, vp, vp, vp, vp, vp, vp]),
            "oq_quantize_weights": (i, [vp, i, i, i, vp, vp, vp, vp, vp, vp]),
            "oq_qlinear": (i, [vp, vp, i, vp, vp, vp, i, vp, i, vp, i, i, vp]),
            "oq_unpack_indices": (i, [vp, i, i, i, vp, vp]),
            "oq_linear_forward_noalloc": (i, [vp, i, i, i, vp, vp, vp, vp, i, vp, vp, i, i, vp]),
            "oq_forward_workspace_bytes": (i, [i, i, i, i, C.POINTER(sz)]),
            "oq_linear_forward_host": (i, [vp, i, i, vp, vp, vp, vp, i, vp, vp, vp, sz, vp]),
            "oq_device_status": (i, [C.POINTER(i)]),
            "oq_selftest_bounded_wait": (i, [vp]),
            "oq_debug_select_rq_kernel": (i, [i]),
            "oq_debug_select_gemm_kernel": (i, [i]),
            "oq_rq_plan": (i, [vp, vp, C.POINTER(i), C.POINTER(i), C.POINTER(i), C.POINTER(sz)]),
            "oq_rotate_quantize_act_levels": (i, [vp, i, i, i, vp, vp, vp, i, vp, vp, vp, vp]),
            "oq_decode_levels": (i, [vp, i, i, vp, vp, i, vp]),
            "oq_qlinear_levels": (i, [vp, i, vp, i, vp, vp, i, vp, i, vp, i, i, vp]),
            "oq_adaln_packed_bytes": (i, [i, i, C.POINTER(sz), C.POINTER(sz)]),
            "oq_adaln_quantize_weights": (i, [vp, i, i, i, vp, vp, vp]),
            "oq_adaln_linear": (i, [vp, i, i, vp, vp, i, i, vp, i, i, vp]),
            "oq_adaln_unpack": (i, [vp, vp, i, i, vp, vp, vp]),
            "oq_block_forward": (i, [i, vp, i, vp, i, vp]),
            "oq_last_error": (C.c_char_p, []), "oq_version": (C.c_char_p, []),
        }
        for name, (res, args) in sig.items():
            if hasattr(L, name):
                f = getattr(L, name)
                f.restype, f.argtypes = res, args
        _lib = L
    return _lib


def _check(code):
    if code != 0:
        raise OqError(code, lib().oq_last_error().decode())


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Codebook:
    """Owns an oq_codebook handle."""

    def __init__(self, dim, bits):
        h = C.c_void_p()
        _check(lib().oq_build_codebook(dim, bits, C.byref(h)))
        self.handle, self.dim, self.bits = h, dim, bits
        L = 1 << bits
        self.centroids = np.zeros(L, np.float64)
        self.boundaries = np.zeros(L - 1, np.float64)
        self.boundaries_f32 = np.zeros(L - 1, np.float32)
        self.centroids_bf16_bits = np.zeros(L, np.uint16)
        _check(lib().oq_codebook_get(h, self.centroids.ctypes.data, self.boundaries.ctypes.data,
                                     self.boundaries_f32.ctypes.data, self.centroids_bf16_bits.ctypes.data))

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.oq_codebook_destroy(self.handle)
            self.handle = None


class Rpbh:
    """Owns an oq_rpbh handle."""

    def __init__(self, dim, block, seed):
        h = C.c_void_p()
        _check(lib().oq_make_rpbh(dim, block, seed, C.byref(h)))
        self.handle, self.dim, self.block, self.seed = h, dim, block, seed
        self.perm = np.zeros(dim, np.int32)
        self.signs = np.zeros(dim, np.int8)
        _check(lib().oq_rpbh_get(h, self.perm.ctypes.data, self.signs.ctypes.data))

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.oq_rpbh_destroy(self.handle)
            self.handle = None


def oq_build_codebook(dim, bits):
    return Codebook(dim, bits)


def oq_make_rpbh(dim, block, seed):
    return Rpbh(dim, block, seed)


def oq_packed_bytes(rows, dim, bits):
    a, b = C.c_size_t(), C.c_size_t()
    _check(lib().oq_packed_bytes(rows, dim, bits, C.byref(a), C.byref(b)))
    return a.value, b.value


def _alloc_packed(rows, dim, bits, device):
    import torch
    total, pitch = oq_packed_bytes(rows, dim, bits)
    return torch.empty((rows, pitch), dtype=torch.uint8, device=device)


def oq_rotate_quantize_act(X, rot, cb_a, out_idx=None, out_norm=None, dbg_rotated=None):
    """X: CUDA bf16 [N, d] (row stride = ldx).  Returns (packed uint8 [N, pitch], norm fp32 [N])."""
    import torch
    n, d = X.shape
    if out_idx is None:
        out_idx = _alloc_packed(n, d, cb_a.bits, X.device)
    if out_norm is None:
        out_norm = torch.empty(n, dtype=torch.float32, device=X.device)
    _check(lib().oq_rotate_quantize_act(_ptr(X), n, d, X.stride(0) if n > 1 else d, rot.handle, cb_a.handle,
                                        _ptr(out_idx), _ptr(out_norm), _ptr(dbg_rotated), _stream()))
    return out_idx, out_norm


def oq_quantize_weights(W, rot, cb_w, out_idx=None, out_norm=None, dbg_rotated=None):
    """W: CUDA bf16 [m, d].  Returns (packed uint8 [m, pitch], row norms bf16 [m])."""
    import torch
    m, d = W.shape
    if out_idx is None:
        out_idx = _alloc_packed(m, d, cb_w.bits, W.device)
    if out_norm is None:
        out_norm = torch.empty(m, dtype=torch.bfloat16, device=W.device)
    _check(lib().oq_quantize_weights(_ptr(W), m, d, W.stride(0) if m > 1 else d, rot.handle, cb_w.handle,
                                     _ptr(out_idx), _ptr(out_norm), _ptr(dbg_rotated), _stream()))
    return out_idx, out_norm


def oq_qlinear(Xq_idx, Xq_norm, cb_a, Wq_idx, Wq_norm, cb_w, dim, out=None, out_dtype=None):
    """Returns Y [N, m] (bf16 by default, fp32 when out_dtype is torch.float32)."""
    import torch
    n, m = Xq_idx.shape[0], Wq_idx.shape[0]
    if out is None:
        out = torch.empty((n, m), dtype=out_dtype or torch.bfloat16, device=Xq_idx.device)
    ydt = OQ_F32 if out.dtype == torch.float32 else OQ_BF16
    _check(lib().oq_qlinear(_ptr(Xq_idx), _ptr(Xq_norm), n, cb_a.handle, _ptr(Wq_idx), _ptr(Wq_norm), m,
                            cb_w.handle, dim, _ptr(out), out.stride(0) if n > 1 else m, ydt, _stream()))
    return out


class _BlockInput(C.Structure):          # oq_block_input
    _fields_ = [("X_bf16", C.c_void_p), ("ldx", C.c_int), ("dim", C.c_int), ("rot", C.c_void_p), ("cb_a", C.c_void_p),
                ("Xq", C.c_void_p), ("Xq_norm", C.c_void_p)]


class _BlockLayer(C.Structure):          # oq_block_layer
    _fields_ = [("input", C.c_int), ("m", C.c_int), ("Wq_idx", C.c_void_p), ("Wq_norm_bf16", C.c_void_p),
                ("cb_w", C.c_void_p), ("Y", C.c_void_p), ("ldy", C.c_int), ("y_dtype", C.c_int)]


def oq_block_forward(inputs, layers):
    """The linear layers of one block on the current stream; every input is rotated and quantized once.
    inputs: list of dicts {X (CUDA bf16 [N, d]), rot, cb_a, xq (scratch: packed uint8 [N, pitch], or bf16 [N, d] at 6 bits),
    xs (fp32 [N])}; layers: list of dicts {input (index), wq, wr, cb_w, Y (CUDA [N, m] bf16 or fp32)}."""
    import torch
    n = inputs[0]["X"].shape[0] if inputs else 0
    ins = (_BlockInput * max(1, len(inputs)))()
    for k, a in enumerate(inputs):
        X = a["X"]
        d = X.shape[1]
        ins[k] = _BlockInput(X.data_ptr(), X.stride(0) if n > 1 else d, d, a["rot"].handle, a["cb_a"].handle,
                             a["xq"].data_ptr(), a["xs"].data_ptr())
    lys = (_BlockLayer * max(1, len(layers)))()
    for k, l in enumerate(layers):
        Y = l["Y"]
        m = Y.shape[1]
        lys[k] = _BlockLayer(l["input"], m, l["wq"].data_ptr(), l["wr"].data_ptr(), l["cb_w"].handle, Y.data_ptr(),
                             Y.stride(0) if n > 1 else m, OQ_F32 if Y.dtype == torch.float32 else OQ_BF16)
    _check(lib().oq_block_forward(n, C.cast(ins, C.c_void_p), len(inputs), C.cast(lys, C.c_void_p), len(layers), _stream()))


def oq_forward_workspace_bytes(n_tokens, dim, m, bits_a):
    b = C.c_size_t()
    _check(lib().oq_forward_workspace_bytes(n_tokens, dim, m, bits_a, C.byref(b)))
    return b.value


def oq_linear_forward_host(X_host, rot, cb_a, Wq_idx, Wq_norm, cb_w, Y_host, workspace):
    """X_host / Y_host: CPU bf16 tensors (pinned for asynchronous copies); workspace: CUDA uint8 tensor."""
    n, d = X_host.shape
    m = Wq_idx.shape[0]
    _check(lib().oq_linear_forward_host(_ptr(X_host), n, d, rot.handle, cb_a.handle, _ptr(Wq_idx), _ptr(Wq_norm), m,
                                        cb_w.handle, _ptr(Y_host), _ptr(workspace), workspace.numel(), _stream()))
    return Y_host


def oq_linear_forward_noalloc(X, rot, cb_a, Wq_idx, Wq_norm, cb_w, out):
    """Allocation-free layer call: X CUDA bf16 [N, d], `out` a preallocated CUDA [N, m] bf16 or fp32 tensor.
    Nothing is allocated here or in the library (the hand-over buffers are a static device array)."""
    import torch
    n, d = X.shape
    m = Wq_idx.shape[0]
    ydt = OQ_F32 if out.dtype == torch.float32 else OQ_BF16
    _check(lib().oq_linear_forward_noalloc(_ptr(X), n, d, X.stride(0) if n > 1 else d, rot.handle, cb_a.handle,
                                           _ptr(Wq_idx), _ptr(Wq_norm), m, cb_w.handle, _ptr(out),
                                           out.stride(0) if n > 1 else m, ydt, _stream()))
    return out


def oq_unpack_indices(idx, rows, dim, bits):
    import torch
    out = torch.empty((rows, dim), dtype=torch.uint8, device=idx.device)
    _check(lib().oq_unpack_indices(_ptr(idx), rows, dim, bits, _ptr(out), _stream()))
    return out


def oq_device_status():
    s = C.c_int(0)
    code = lib().oq_device_status(C.byref(s))
    if code not in (0, 5):
        _check(code)
    return s.value


def oq_selftest_bounded_wait():
    _check(lib().oq_selftest_bounded_wait(_stream()))


def oq_rq_plan(rot, cb):
    """(kernel, rows_per_group, tiles_per_group, smem_bytes) of the rotate+quantize launch for these handles."""
    k, r, t, m = C.c_int(0), C.c_int(0), C.c_int(0), C.c_size_t(0)
    _check(lib().oq_rq_plan(rot.handle, cb.handle, C.byref(k), C.byref(r), C.byref(t), C.byref(m)))
    return k.value, r.value, t.value, m.value


def oq_debug_select_rq_kernel(which):
    _check(lib().oq_debug_select_rq_kernel(int(which)))


def oq_debug_select_gemm_kernel(which):
    _check(lib().oq_debug_select_gemm_kernel(int(which)))


def oq_rotate_quantize_act_levels(X, rot, cb_a, out=None, out_norm=None, want_idx=False, dbg_rotated=None):
    """6-bit activations: X CUDA bf16 [N, d] -> (levels bf16 [N, d], norm fp32 [N], idx uint8 [N, d] or None)."""
    import torch
    n, d = X.shape
    if out is None:
        out = torch.empty((n, d), dtype=torch.bfloat16, device=X.device)
    if out_norm is None:
        out_norm = torch.empty(n, dtype=torch.float32, device=X.device)
    idx = torch.empty((n, d), dtype=torch.uint8, device=X.device) if want_idx else None
    _check(lib().oq_rotate_quantize_act_levels(_ptr(X), n, d, X.stride(0) if n > 1 else d, rot.handle, cb_a.handle,
                                               _ptr(out), out.stride(0) if n > 1 else d, _ptr(out_norm), _ptr(idx),
                                               _ptr(dbg_rotated), _stream()))
    return out, out_norm, idx


def oq_decode_levels(idx, rows, dim, cb, out=None):
    """Packed indices [rows, pitch] -> bf16 levels [rows, dim] (written once, read by oq_qlinear_levels)."""
    import torch
    if out is None:
        out = torch.empty((rows, dim), dtype=torch.bfloat16, device=idx.device)
    _check(lib().oq_decode_levels(_ptr(idx), rows, dim, cb.handle, _ptr(out), out.stride(0) if rows > 1 else dim, _stream()))
    return out


def oq_qlinear_levels(Xd, Xq_norm, Wq_idx, Wq_norm, cb_w, dim, out=None, out_dtype=None):
    """oq_qlinear with the activations given as bf16 levels [N, dim]."""
    import torch
    n, m = Xd.shape[0], Wq_idx.shape[0]
    if out is None:
        out = torch.empty((n, m), dtype=out_dtype or torch.bfloat16, device=Xd.device)
    ydt = OQ_F32 if out.dtype == torch.float32 else OQ_BF16
    _check(lib().oq_qlinear_levels(_ptr(Xd), Xd.stride(0) if n > 1 else dim, _ptr(Xq_norm), n, _ptr(Wq_idx),
                                   _ptr(Wq_norm), m, cb_w.handle, dim, _ptr(out), out.stride(0) if n > 1 else m, ydt,
                                   _stream()))
    return out


def oq_adaln_packed_bytes(m, dim):
    a, b = C.c_size_t(), C.c_size_t()
    _check(lib().oq_adaln_packed_bytes(m, dim, C.byref(a), C.byref(b)))
    return a.value, b.value


def oq_adaln_quantize_weights(W):
    """W: CUDA bf16 [m, d].  Returns (packed nibbles uint8 [m * d / 2], scales uint8 [2 * m * d / 64])."""
    import torch
    m, d = W.shape
    wq_bytes, sc_bytes = oq_adaln_packed_bytes(m, d)
    Wq = torch.empty(wq_bytes, dtype=torch.uint8, device=W.device)
    Sc = torch.empty(sc_bytes, dtype=torch.uint8, device=W.device)
    _check(lib().oq_adaln_quantize_weights(_ptr(W), m, d, W.stride(0) if m > 1 else d, _ptr(Wq), _ptr(Sc), _stream()))
    return Wq, Sc


def oq_adaln_linear(X, Wq, Sc, m, out=None, out_dtype=None):
    """X: CUDA bf16 [n, d].  Returns Y [n, m] (bf16 by default, fp32 when out_dtype is torch.float32)."""
    import torch
    n, d = X.shape
    if out is None:
        out = torch.empty((n, m), dtype=out_dtype or torch.bfloat16, device=X.device)
    ydt = OQ_F32 if out.dtype == torch.float32 else OQ_BF16
    _check(lib().oq_adaln_linear(_ptr(X), n, X.stride(0) if n > 1 else d, _ptr(Wq), _ptr(Sc), m, d, _ptr(out),
                                 out.stride(0) if n > 1 else m, ydt, _stream()))
    return out


def oq_adaln_unpack(Wq, Sc, m, dim):
    """Returns (q int8 [m, d], scale bf16 [m, d / 64]) on the device."""
    import torch
    q = torch.empty((m, dim), dtype=torch.int8, device=Wq.device)
    s = torch.empty((m, dim // 64), dtype=torch.bfloat16, device=Wq.device)
    _check(lib().oq_adaln_unpack(_ptr(Wq), _ptr(Sc), m, dim, _ptr(q), _ptr(s), _stream()))
    return q, s


def oq_version():
    return lib().oq_version().decode()
