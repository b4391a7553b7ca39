"""ctypes binding of ``libautoassist.so`` — argument marshalling only.

Every step of the path runs in the CUDA library; this module turns torch tensors into the
plain pointers and sizes of ``include/autoassist.h`` and raises on any non-zero status.
There is no fallback: if the library has not been built, loading fails with an error.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_float, c_int32, c_int64, c_size_t, c_uint64, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libautoassist.so")

AA_OK = 0
AA_ERR_INVALID_ARG, AA_ERR_UNSUPPORTED, AA_ERR_CUDA, AA_ERR_WORKSPACE = 1, 2, 3, 4
AA_ERR_SCAN_TIMEOUT, AA_ERR_BAD_INDEX, AA_ERR_CAPACITY = 5, 6, 7
AA_F32, AA_BF16 = 0, 1
AA_FEAT_DENSE, AA_FEAT_CSR = 0, 1
AA_ASSIST_LINEAR, AA_ASSIST_MLP = 0, 1
AA_THRESH_VALUE, AA_THRESH_BATCH_MEAN = 0, 1

EXPORTS = (
    "aa_status_string", "aa_workspace_bytes", "aa_create", "aa_destroy", "aa_score_shrink",
    "aa_shrink_compact", "aa_instance_loss", "aa_assistant_step", "aa_step_host_staging_bytes", "aa_step_host",
    "aa_device_status", "aa_launch_count", "aa_shrink_compact_static", "aa_batch_cut", "aa_threshold_compact", "aa_sk_threshold", "aa_assistant_step_adam",
    "aa_instance_loss_rows", "aa_assistant_step_scored", "aa_conv_pool_features",
)
AA_STATIC_MAX_CANDIDATES = 1 << 22


class aa_feat(Structure):
    _fields_ = [
        ("kind", c_int32), ("dtype", c_int32), ("n", c_int64), ("d", c_int64),
        ("dense", c_void_p), ("row_stride", c_int64),
        ("indptr", c_void_p), ("col", c_void_p), ("val", c_void_p), ("nnz", c_int64),
        ("row_idx", c_void_p), ("n_rows", c_int64), ("id_base", c_int64),
    ]


class aa_assistant(Structure):
    _fields_ = [
        ("kind", c_int32), ("reserved", c_int32), ("d", c_int64), ("hidden", c_int64),
        ("w", c_void_p), ("b", c_void_p),
        ("W1", c_void_p), ("W1_bf16", c_void_p), ("b1", c_void_p), ("w2", c_void_p), ("b2", c_void_p),
    ]


class aa_logits(Structure):
    _fields_ = [
        ("data", c_void_p), ("dtype", c_int32), ("reserved", c_int32),
        ("rows", c_int64), ("cols", c_int64), ("row_stride", c_int64),
    ]


class aa_conv(Structure):
    _fields_ = [("c_in", c_int32), ("height", c_int32), ("width", c_int32), ("c_out", c_int32), ("ksize", c_int32), ("pool", c_int32),
                ("weight", c_void_p), ("bias", c_void_p)]


def conv_layer(weight: torch.Tensor, bias, height: int, width: int, pool: int) -> aa_conv:
    """The Boss's convolution for the convolutional Assistant: weight fp32 [c_out, c_in, k, k], bias fp32 [c_out] or None."""
    _check(weight, torch.float32, "weight")
    _check(bias, torch.float32, "bias")
    if weight.dim() != 4 or weight.shape[2] != weight.shape[3]:
        raise TypeError("weight must be [c_out, c_in, k, k]")
    cv = aa_conv()
    cv.c_out, cv.c_in, cv.ksize = weight.shape[0], weight.shape[1], weight.shape[2]
    cv.height, cv.width, cv.pool = height, width, pool
    cv.weight, cv.bias = weight.data_ptr(), _ptr(bias)
    cv._keep = (weight, bias)
    return cv


class aa_adam(Structure):
    _fields_ = [("beta1", c_float), ("beta2", c_float), ("eps", c_float), ("reserved", c_int32), ("t", c_int64),
                ("m", c_void_p), ("v", c_void_p)]


def adam_state(m: torch.Tensor, v: torch.Tensor, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8) -> aa_adam:
    """Adam moments (fp32 device tensors laid out like the flattened parameters, zero before the first step)."""
    _check(m, torch.float32, "m")
    _check(v, torch.float32, "v")
    st = aa_adam()
    st.beta1, st.beta2, st.eps, st.t = beta1, beta2, eps, 0
    st.m, st.v = m.data_ptr(), v.data_ptr()
    st._keep = (m, v)
    return st


class AutoAssistError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (aa_status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """The CUDA library; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1905_03381_b200.build` "
                "(nvcc, sm_100a). The library has no CPU or PyTorch fallback."
            )
        L = ctypes.CDLL(LIB_PATH)
        L.aa_status_string.restype = ctypes.c_char_p
        L.aa_status_string.argtypes = [c_int32]
        L.aa_workspace_bytes.argtypes = [c_int64, c_int64, c_int64, POINTER(c_size_t)]
        L.aa_create.argtypes = [POINTER(c_void_p), c_int64, c_int64, c_int64, c_void_p, c_size_t, c_void_p]
        L.aa_destroy.argtypes = [c_void_p]
        L.aa_score_shrink.argtypes = [c_void_p, POINTER(aa_feat), POINTER(aa_assistant), c_float, c_uint64, c_uint64,
                                      c_void_p, c_int64, c_void_p, c_void_p, c_void_p]
        L.aa_shrink_compact.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_float, c_uint64, c_uint64,
                                        c_void_p, c_int64, c_void_p, c_void_p]
        L.aa_shrink_compact_static.argtypes = [c_void_p, c_int64, c_int64, c_float, c_uint64, c_uint64,
                                               c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]
        L.aa_assistant_step_adam.argtypes = [c_void_p, POINTER(aa_feat), c_void_p, c_void_p, POINTER(aa_assistant),
                                             POINTER(aa_adam), c_float, c_int32, c_float]
        L.aa_threshold_compact.argtypes = [c_void_p, c_void_p, c_int64, c_float, c_void_p, c_int64, c_void_p, c_void_p]
        L.aa_sk_threshold.restype = c_float
        L.aa_sk_threshold.argtypes = [c_float, c_int64]
        L.aa_batch_cut.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_int64, c_int64,
                                   c_void_p, c_void_p, c_void_p, c_int64]
        L.aa_instance_loss.argtypes = [c_void_p, POINTER(aa_logits), c_void_p, c_void_p, c_int64, c_void_p, c_void_p]
        L.aa_instance_loss_rows.argtypes = [c_void_p, POINTER(aa_logits), c_void_p, c_void_p, c_int64, c_void_p, c_void_p]
        L.aa_assistant_step.argtypes = [c_void_p, POINTER(aa_feat), c_void_p, c_void_p, POINTER(aa_assistant),
                                        c_float, c_int32, c_float]
        L.aa_assistant_step_scored.argtypes = [c_void_p, POINTER(aa_feat), c_void_p, c_void_p, c_void_p, POINTER(aa_assistant),
                                               c_float, c_int32, c_float]
        L.aa_conv_pool_features.argtypes = [c_void_p, POINTER(aa_feat), POINTER(aa_conv), c_void_p, c_int64]
        L.aa_step_host_staging_bytes.argtypes = [POINTER(aa_feat), POINTER(aa_logits), POINTER(c_size_t)]
        L.aa_step_host.argtypes = [c_void_p, POINTER(aa_feat), POINTER(aa_assistant), c_float, c_uint64, c_uint64,
                                   POINTER(aa_logits), c_void_p, c_float, c_int32, c_float,
                                   c_void_p, c_void_p, c_void_p, c_void_p, c_size_t]
        L.aa_device_status.argtypes = [c_void_p, POINTER(c_int32)]
        L.aa_launch_count.restype = c_int64
        L.aa_launch_count.argtypes = [c_void_p]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().aa_status_string(status).decode()


def aa_shrink_compact_static(score: torch.Tensor, mix: float, seed: int, step: int, out_idx: torch.Tensor,
                             out_count: torch.Tensor, out_mask=None, out_status=None, id_base: int = 0, n=None,
                             stream=None):
    """Shrink + compact on precomputed scores with no context and no workspace: the scan state is a fixed
    array inside the library (for callers that cannot allocate device memory).  At most
    AA_STATIC_MAX_CANDIDATES scores per call; calls on one device must not overlap."""
    with torch.cuda.device(score.device):
        s = stream if stream is not None else torch.cuda.current_stream(score.device)
        st = lib().aa_shrink_compact_static(score.data_ptr(), score.numel() if n is None else n, id_base, mix, seed,
                                            step, out_idx.data_ptr(), out_idx.numel(), out_count.data_ptr(),
                                            _ptr(out_mask), _ptr(out_status), s.cuda_stream)
    if st != AA_OK:
        raise AutoAssistError(st, "aa_shrink_compact_static")


def aa_sk_threshold(G: float, k: int) -> float:
    """T_k = G / k, the shrinking threshold schedule of the paper's convergence theorem."""
    return float(lib().aa_sk_threshold(G, k))


def _ptr(t):
    return None if t is None else t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return AA_F32
    if t.dtype == torch.bfloat16:
        return AA_BF16
    raise TypeError(f"expected float32 or bfloat16, got {t.dtype}")


def _check(t, dtype, name):
    if t is not None and (t.dtype != dtype or not t.is_cuda or not t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor of {dtype}")


def dense_features(x: torch.Tensor, row_idx=None, n_rows=None, id_base: int = 0) -> aa_feat:
    """Descriptor of a row-major [n, d] fp32/bf16 matrix (last dim contiguous; row stride free)."""
    if x.dim() != 2 or x.stride(1) != 1 or not x.is_cuda:
        raise TypeError("x must be a 2-D CUDA tensor with contiguous rows")
    _check(row_idx, torch.int32, "row_idx")
    f = aa_feat()
    f.kind, f.dtype, f.n, f.d = AA_FEAT_DENSE, _dtype_code(x), x.shape[0], x.shape[1]
    f.dense, f.row_stride = x.data_ptr(), x.stride(0) if x.shape[0] > 1 else x.shape[1]
    f.row_idx = _ptr(row_idx)
    f.n_rows = 0 if row_idx is None else (row_idx.numel() if n_rows is None else n_rows)
    f.id_base = id_base
    f._keep = (x, row_idx)
    return f


def csr_features(indptr, col, val, d: int, nnz=None, row_idx=None, n_rows=None, id_base: int = 0) -> aa_feat:
    """Descriptor of CSR rows: indptr[n+1] int32, col[nnz] int32 in [0, d), val[nnz] fp32."""
    _check(indptr, torch.int32, "indptr")
    _check(col, torch.int32, "col")
    _check(val, torch.float32, "val")
    _check(row_idx, torch.int32, "row_idx")
    f = aa_feat()
    f.kind, f.dtype, f.n, f.d = AA_FEAT_CSR, AA_F32, indptr.numel() - 1, d
    f.indptr, f.col, f.val = indptr.data_ptr(), _ptr(col), _ptr(val)
    f.nnz = col.numel() if nnz is None else nnz
    f.row_idx = _ptr(row_idx)
    f.n_rows = 0 if row_idx is None else (row_idx.numel() if n_rows is None else n_rows)
    f.id_base = id_base
    f._keep = (indptr, col, val, row_idx)
    return f


def linear_assistant(w: torch.Tensor, b: torch.Tensor) -> aa_assistant:
    _check(w, torch.float32, "w")
    _check(b, torch.float32, "b")
    a = aa_assistant()
    a.kind, a.d, a.hidden = AA_ASSIST_LINEAR, w.numel(), 0
    a.w, a.b = w.data_ptr(), b.data_ptr()
    a._keep = (w, b)
    return a


def mlp_assistant(W1: torch.Tensor, W1_bf16: torch.Tensor, b1: torch.Tensor, w2: torch.Tensor, b2: torch.Tensor) -> aa_assistant:
    """Two-layer Assistant: W1 fp32 master [hidden, d], its bf16 copy, b1[hidden], w2[hidden], b2[1]."""
    for t, name in ((W1, "W1"), (b1, "b1"), (w2, "w2"), (b2, "b2")):
        _check(t, torch.float32, name)
    _check(W1_bf16, torch.bfloat16, "W1_bf16")
    if W1.dim() != 2 or W1_bf16.shape != W1.shape or b1.numel() != W1.shape[0] or w2.numel() != W1.shape[0]:
        raise TypeError("W1 must be [hidden, d] with matching W1_bf16, b1[hidden], w2[hidden]")
    a = aa_assistant()
    a.kind, a.hidden, a.d = AA_ASSIST_MLP, W1.shape[0], W1.shape[1]
    a.W1, a.W1_bf16, a.b1, a.w2, a.b2 = W1.data_ptr(), W1_bf16.data_ptr(), b1.data_ptr(), w2.data_ptr(), b2.data_ptr()
    a._keep = (W1, W1_bf16, b1, w2, b2)
    return a


def logits_desc(logits: torch.Tensor, rows=None) -> aa_logits:
    if logits.dim() != 2 or logits.stride(1) != 1 or not logits.is_cuda:
        raise TypeError("logits must be a 2-D CUDA tensor with contiguous rows")
    g = aa_logits()
    g.data, g.dtype = logits.data_ptr(), _dtype_code(logits)
    g.rows = logits.shape[0] if rows is None else rows
    g.cols = logits.shape[1]
    g.row_stride = logits.stride(0) if logits.shape[0] > 1 else logits.shape[1]
    g._keep = logits
    return g


class AutoAssist:
    """One library context: a workspace tensor, a CUDA stream, and the C entry points as methods."""

    def __init__(self, max_rows: int, max_d: int, max_hidden: int = 0, device="cuda:0", stream=None):
        L = lib()
        self.device = torch.device(device)
        nbytes = c_size_t(0)
        self._ok(L.aa_workspace_bytes(max_rows, max_d, max_hidden, byref(nbytes)), "aa_workspace_bytes")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self._ctx = c_void_p()
            self._ok(L.aa_create(byref(self._ctx), max_rows, max_d, max_hidden, self._ws_ptr, nbytes.value,
                                 self.stream.cuda_stream), "aa_create")
        self._L = L

    @staticmethod
    def _ok(status: int, where: str):
        if status != AA_OK:
            raise AutoAssistError(status, where)

    def close(self):
        if getattr(self, "_ctx", None):
            self._L.aa_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def aa_score_shrink(self, feat: aa_feat, assistant: aa_assistant, mix: float, seed: int, step: int,
                        out_idx: torch.Tensor, out_count: torch.Tensor, out_score=None, out_mask=None):
        self._ok(self._L.aa_score_shrink(self._ctx, byref(feat), byref(assistant), mix, seed, step,
                                         out_idx.data_ptr(), out_idx.numel(), out_count.data_ptr(),
                                         _ptr(out_score), _ptr(out_mask)), "aa_score_shrink")

    def aa_shrink_compact(self, score: torch.Tensor, mix: float, seed: int, step: int, out_idx: torch.Tensor,
                          out_count: torch.Tensor, out_mask=None, id_base: int = 0, n=None):
        self._ok(self._L.aa_shrink_compact(self._ctx, score.data_ptr(), score.numel() if n is None else n, id_base,
                                           mix, seed, step, out_idx.data_ptr(), out_idx.numel(),
                                           out_count.data_ptr(), _ptr(out_mask)), "aa_shrink_compact")

    def aa_threshold_compact(self, value: torch.Tensor, threshold: float, out_idx: torch.Tensor, out_count: torch.Tensor,
                             out_mask=None, n=None):
        """Hard shrinking: ordered list of the instances whose value (loss or gradient magnitude) is >= threshold."""
        _check(value, torch.float32, "value")
        self._ok(self._L.aa_threshold_compact(self._ctx, value.data_ptr(), value.numel() if n is None else n, threshold,
                                              out_idx.data_ptr(), out_idx.numel(), out_count.data_ptr(), _ptr(out_mask)),
                 "aa_threshold_compact")

    def aa_batch_cut(self, idx: torch.Tensor, count_dev: torch.Tensor, n_cand: int, out_m: torch.Tensor,
                     out_consumed: torch.Tensor, batch_size: int = 0, lengths=None, token_budget: int = 0, out_offsets=None):
        """The batch Algorithm 1 returns (first batch_size survivors, or the longest prefix within a token budget) and
        how many candidates its walk covered; all results stay on the device."""
        _check(lengths, torch.int32, "lengths")
        _check(out_offsets, torch.int32, "out_offsets")
        self._ok(self._L.aa_batch_cut(self._ctx, idx.data_ptr(), _ptr(count_dev), idx.numel(), n_cand, batch_size,
                                      _ptr(lengths), 0 if lengths is None else lengths.numel(), token_budget,
                                      out_m.data_ptr(), out_consumed.data_ptr(), _ptr(out_offsets),
                                      0 if out_offsets is None else out_offsets.numel()), "aa_batch_cut")

    def aa_instance_loss(self, logits: aa_logits, labels: torch.Tensor, out_loss: torch.Tensor, offsets=None,
                         n_seg=None, count_dev=None):
        if offsets is not None and n_seg is None:
            n_seg = offsets.numel() - 1
        self._ok(self._L.aa_instance_loss(self._ctx, byref(logits), labels.data_ptr(), _ptr(offsets),
                                          0 if n_seg is None else n_seg, _ptr(count_dev), out_loss.data_ptr()),
                 "aa_instance_loss")

    def aa_instance_loss_rows(self, logits: aa_logits, labels: torch.Tensor, row_idx: torch.Tensor, out_loss: torch.Tensor,
                              count_dev=None, n_rows=None):
        """Losses of the batch instances row_idx[k] out of logits / labels stored for the whole pool."""
        _check(row_idx, torch.int32, "row_idx")
        self._ok(self._L.aa_instance_loss_rows(self._ctx, byref(logits), labels.data_ptr(), row_idx.data_ptr(),
                                               row_idx.numel() if n_rows is None else n_rows, _ptr(count_dev),
                                               out_loss.data_ptr()), "aa_instance_loss_rows")

    def aa_assistant_step(self, feat: aa_feat, loss: torch.Tensor, assistant: aa_assistant, lr: float,
                          threshold=None, count_dev=None):
        """threshold=None labels against the batch mean loss."""
        mode = AA_THRESH_BATCH_MEAN if threshold is None else AA_THRESH_VALUE
        self._ok(self._L.aa_assistant_step(self._ctx, byref(feat), loss.data_ptr(), _ptr(count_dev), byref(assistant),
                                           lr, mode, 0.0 if threshold is None else threshold), "aa_assistant_step")

    def aa_assistant_step_scored(self, feat: aa_feat, loss: torch.Tensor, score: torch.Tensor, assistant: aa_assistant, lr: float,
                                 threshold=None, count_dev=None):
        """aa_assistant_step with the pre-activations that screening wrote (out_score, one per stored row): valid only
        while the parameters are those the pool was screened with.  The two-layer Assistant also takes the gates that
        the last screening on this context left in its workspace (same pool, same W1_bf16, no update in between);
        otherwise it evaluates the forward pass itself."""
        _check(score, torch.float32, "score")
        mode = AA_THRESH_BATCH_MEAN if threshold is None else AA_THRESH_VALUE
        self._ok(self._L.aa_assistant_step_scored(self._ctx, byref(feat), loss.data_ptr(), _ptr(count_dev), _ptr(score),
                                                  byref(assistant), lr, mode, 0.0 if threshold is None else threshold),
                 "aa_assistant_step_scored")

    def aa_conv_pool_features(self, images: aa_feat, conv: aa_conv, out_phi: torch.Tensor):
        """phi = average-pooled, rectified convolution of every stored image row (the convolutional Assistant's first
        two layers); out_phi is an fp32 [n, c_out * (height // pool) * (width // pool)] CUDA tensor with contiguous rows."""
        if out_phi.dtype != torch.float32 or out_phi.dim() != 2 or out_phi.stride(1) != 1 or not out_phi.is_cuda:
            raise TypeError("out_phi must be a 2-D fp32 CUDA tensor with contiguous rows")
        self._ok(self._L.aa_conv_pool_features(self._ctx, byref(images), byref(conv), out_phi.data_ptr(),
                                               out_phi.stride(0) if out_phi.shape[0] > 1 else out_phi.shape[1]),
                 "aa_conv_pool_features")

    def aa_assistant_step_adam(self, feat: aa_feat, loss: torch.Tensor, assistant: aa_assistant, state: aa_adam, lr: float,
                               threshold=None, count_dev=None):
        """aa_assistant_step with Adam; state.t advances."""
        mode = AA_THRESH_BATCH_MEAN if threshold is None else AA_THRESH_VALUE
        self._ok(self._L.aa_assistant_step_adam(self._ctx, byref(feat), loss.data_ptr(), _ptr(count_dev), byref(assistant),
                                                byref(state), lr, mode, 0.0 if threshold is None else threshold),
                 "aa_assistant_step_adam")

    def host_step_plan(self, x_host: torch.Tensor, logits_host: torch.Tensor):
        """Descriptors and a device staging buffer for aa_step_host on HOST tensors of these shapes."""
        f = aa_feat()
        f.kind, f.dtype, f.n, f.d = AA_FEAT_DENSE, _dtype_code(x_host), x_host.shape[0], x_host.shape[1]
        f.dense, f.row_stride = x_host.data_ptr(), x_host.shape[1]
        g = aa_logits()
        g.data, g.dtype = logits_host.data_ptr(), _dtype_code(logits_host)
        g.rows, g.cols, g.row_stride = logits_host.shape[0], logits_host.shape[1], logits_host.shape[1]
        nbytes = c_size_t(0)
        self._ok(self._L.aa_step_host_staging_bytes(byref(f), byref(g), byref(nbytes)), "aa_step_host_staging_bytes")
        staging = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        f._keep, g._keep = x_host, logits_host
        return f, g, staging, nbytes.value

    def aa_step_host(self, feat: aa_feat, assistant: aa_assistant, mix: float, seed: int, step: int, logits: aa_logits,
                     labels_host: torch.Tensor, lr: float, out_idx_host: torch.Tensor, out_count_host: torch.Tensor,
                     out_loss_host: torch.Tensor, staging: torch.Tensor, staging_bytes: int, threshold=None):
        """Whole step on HOST buffers (features, logits, labels in; batch list, count, losses out)."""
        mode = AA_THRESH_BATCH_MEAN if threshold is None else AA_THRESH_VALUE
        sp = (staging.data_ptr() + 255) // 256 * 256
        self._ok(self._L.aa_step_host(self._ctx, byref(feat), byref(assistant), mix, seed, step, byref(logits),
                                      labels_host.data_ptr(), lr, mode, 0.0 if threshold is None else threshold,
                                      out_idx_host.data_ptr(), out_count_host.data_ptr(), out_loss_host.data_ptr(),
                                      sp, staging_bytes), "aa_step_host")

    def aa_device_status(self) -> int:
        latched = c_int32(0)
        self._ok(self._L.aa_device_status(self._ctx, byref(latched)), "aa_device_status")
        return latched.value

    def aa_launch_count(self) -> int:
        return int(self._L.aa_launch_count(self._ctx))
