"""ctypes binding of the C ABI declared in ``include/ssd.h`` (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libssd.so")

SSD_OK, SSD_ERR_BAD_ARG, SSD_ERR_NOT_LOADED, SSD_ERR_INVALID_TREE, SSD_ERR_CTX_OVERFLOW = 0, -1, -2, -3, -4
SSD_ERR_BAD_PATH, SSD_ERR_CUDA, SSD_ERR_TIMEOUT, SSD_ERR_NOMEM, SSD_ERR_UNSUPPORTED = -5, -6, -7, -8, -9
SSD_GREEDY, SSD_SAMPLING = 0, 1
SSD_DTYPE_F32, SSD_DTYPE_BF16, SSD_DTYPE_BF16_W8 = 0, 1, 2
SSD_TUNE_LOW_PLANE, SSD_TUNE_DEPENDENT_LAUNCH, SSD_TUNE_GRAPH, SSD_TUNE_GEMM_CTAS, SSD_TUNE_CLUSTER_REDUCE, SSD_TUNE_CLUSTER_MAX = 0, 1, 2, 3, 4, 5
SSD_TUNE_ATTN_LOW_PLANE, SSD_TUNE_HEAD_CTAS, SSD_TUNE_KERNEL_TRACE = 6, 7, 8
SSD_TUNE_CLUSTER_QKV, SSD_TUNE_CLUSTER_O, SSD_TUNE_CLUSTER_FC, SSD_TUNE_CLUSTER_PROJ, SSD_TUNE_HEAD_STATS = 9, 10, 11, 12, 13
SSD_TUNE_W8_PLANES, SSD_TUNE_STAGE_KV_FROM, SSD_TUNE_ATTN_SPLITS, SSD_TUNE_NODE_GROUPS, SSD_TUNE_FUSED_GELU, SSD_TUNE_ATTN_STAGED_WARPS = 14, 15, 16, 17, 18, 19

# every symbol include/ssd.h declares
EXPORTS = ("ssd_create", "ssd_load_weights", "ssd_w8_read", "ssd_kv_create", "ssd_kv_reset", "ssd_kv_len", "ssd_kv_rollback",
           "ssd_kv_destroy", "ssd_verify_tree", "ssd_accept_tree", "ssd_accept_tree_sparse", "ssd_propose_children", "ssd_kv_commit", "ssd_kv_read", "ssd_strerror",
           "ssd_last_device_status", "ssd_reset_device_status", "ssd_debug_expire_wait", "ssd_last_cuda_error", "ssd_last_cuda_error_line", "ssd_kernel_launches", "ssd_set_tuning", "ssd_get_phase_trace", "ssd_accept_tree_noalloc", "ssd_destroy",
           "ssd_trigram_build", "ssd_trigram_lookup", "ssd_trigram_propose", "ssd_trigram_contexts", "ssd_trigram_destroy")


class ssd_config(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_layer", "d_model", "n_head", "d_head", "d_ff", "vocab", "n_ctx",
                                         "max_nodes", "dtype")] + [("ln_eps", C.c_float)]


class ssd_sampling(C.Structure):
    _fields_ = [("mode", C.c_int32), ("temperature", C.c_float), ("top_k", C.c_int32)]


class ssd_rng(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("step", C.c_uint64)]


_VP = C.c_void_p
_VPP = C.POINTER(C.c_void_p)
_PER_LAYER = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_g", "ln2_b", "w_fc", "b_fc", "w_proj", "b_proj")


class ssd_weights(C.Structure):
    _fields_ = [(k, _VP) for k in ("wte", "wpe", "lnf_g", "lnf_b")] + [(k, _VPP) for k in _PER_LAYER]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def lib():
    """The loaded shared library.  Raises if it has not been built: the product has no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("libssd.so is not built; run `python -m paper_2308_04623_b200.build` "
                              "(nvcc, sm_100a).  There is no CPU fallback.")
        L = C.CDLL(_LIB_PATH)
        L.ssd_create.argtypes = [C.POINTER(ssd_config), C.c_int, _VP, C.POINTER(_VP)]
        L.ssd_load_weights.argtypes = [_VP, C.POINTER(ssd_weights)]
        L.ssd_w8_read.argtypes = [_VP, C.c_int32, C.c_int32, _VP, _VP]
        L.ssd_kv_create.argtypes = [_VP, C.POINTER(_VP)]
        L.ssd_kv_reset.argtypes = [_VP]
        L.ssd_kv_len.argtypes = [_VP, C.POINTER(C.c_int32)]
        L.ssd_kv_rollback.argtypes = [_VP, C.c_int32]
        L.ssd_kv_destroy.argtypes = [_VP]
        L.ssd_kv_destroy.restype = None
        L.ssd_verify_tree.argtypes = [_VP, _VP, _VP, C.c_int32, _VP, _VP]
        L.ssd_accept_tree.argtypes = [_VP, _VP, _VP, _VP, _VP, C.c_int32, C.POINTER(ssd_sampling), C.POINTER(ssd_rng),
                                      _VP, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.ssd_accept_tree_noalloc.argtypes = [C.c_int, _VP, _VP, _VP, _VP, _VP, C.c_int32, C.c_int32, C.POINTER(ssd_sampling),
                                              C.POINTER(ssd_rng), _VP, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.ssd_kv_commit.argtypes = [_VP, _VP, _VP, C.c_int32]
        L.ssd_accept_tree_sparse.argtypes = [_VP, _VP, _VP, _VP, C.c_int32, _VP, _VP, C.c_int32, C.POINTER(ssd_sampling), C.POINTER(ssd_rng),
                                             _VP, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.ssd_propose_children.argtypes = [_VP, _VP, _VP, C.c_int32, C.c_int32, C.POINTER(ssd_sampling), C.POINTER(ssd_rng), _VP, _VP]
        L.ssd_kv_read.argtypes = [_VP, _VP, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _VP]
        L.ssd_strerror.argtypes = [C.c_int]
        L.ssd_strerror.restype = C.c_char_p
        L.ssd_last_device_status.argtypes = [_VP, C.POINTER(C.c_int32)]
        L.ssd_last_cuda_error.argtypes = [_VP]
        L.ssd_last_cuda_error_line.argtypes = [_VP]
        L.ssd_kernel_launches.argtypes = [_VP, C.POINTER(C.c_int64)]
        L.ssd_reset_device_status.argtypes = [_VP]
        L.ssd_debug_expire_wait.argtypes = [_VP, C.c_int32]
        L.ssd_set_tuning.argtypes = [_VP, C.c_int32, C.c_int32]
        L.ssd_get_phase_trace.argtypes = [_VP, _VP, C.c_int32, C.POINTER(C.c_int32)]
        L.ssd_destroy.argtypes = [_VP]
        L.ssd_destroy.restype = None
        L.ssd_trigram_build.argtypes = [_VP, C.c_int64, C.c_int32, C.c_int, _VP, C.POINTER(_VP)]
        L.ssd_trigram_lookup.argtypes = [_VP, _VP, C.c_int32, _VP, _VP]
        L.ssd_trigram_propose.argtypes = [_VP, C.c_int32, C.c_int32, _VP, C.c_int32, _VP, _VP]
        L.ssd_trigram_contexts.argtypes = [_VP, C.POINTER(C.c_int64)]
        L.ssd_trigram_destroy.argtypes = [_VP]
        L.ssd_trigram_destroy.restype = None
        _lib = L
    return _lib


class SsdError(RuntimeError):
    def __init__(self, code: int, cuda: int = 0, line: int = 0):
        msg = lib().ssd_strerror(code).decode()
        super().__init__("libssd: %s (%d)%s" % (msg, code, " cudaError %d at ssd_api.cu:%d" % (cuda, line) if cuda else ""))
        self.code = code
        self.cuda = cuda


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


class Context:
    """ssd_ctx: one model on one device and stream."""

    def __init__(self, cfg: dict, device: int = 0, stream: int = 0):
        self.cfg = dict(cfg)
        c = ssd_config(cfg["n_layer"], cfg["d_model"], cfg["n_head"], cfg["d_head"], cfg["d_ff"], cfg["vocab"],
                       cfg["n_ctx"], cfg["max_nodes"], {"fp32": SSD_DTYPE_F32, "bf16": SSD_DTYPE_BF16, "bf16_w8": SSD_DTYPE_BF16_W8}[cfg["dtype"]], float(cfg["ln_eps"]))
        h = _VP()
        rc = lib().ssd_create(C.byref(c), device, _VP(stream), C.byref(h))
        if rc != SSD_OK:
            raise SsdError(rc)
        self.h = h

    def _chk(self, rc):
        if rc != SSD_OK:
            raise SsdError(rc, lib().ssd_last_cuda_error(self.h), lib().ssd_last_cuda_error_line(self.h))

    def close(self):
        if getattr(self, "h", None):
            lib().ssd_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def load_weights(self, weights: dict):
        """ssd_load_weights.  ``weights``: numpy arrays, float32 for an fp32 model, uint16 bf16 bit
        patterns for a bf16 model; per-layer entries are lists of n_layer arrays."""
        want = np.float32 if self.cfg["dtype"] == "fp32" else np.uint16
        keep, w = [], ssd_weights()
        for k in ("wte", "wpe", "lnf_g", "lnf_b"):
            a = np.ascontiguousarray(weights[k])
            assert a.dtype == want, (k, a.dtype)
            keep.append(a)
            setattr(w, k, a.ctypes.data)
        for k in _PER_LAYER:
            arrs = [np.ascontiguousarray(t) for t in weights[k]]
            assert all(t.dtype == want for t in arrs), k
            keep.extend(arrs)
            tab = (_VP * len(arrs))(*[t.ctypes.data for t in arrs])
            keep.append(tab)
            setattr(w, k, C.cast(tab, _VPP))
        self._chk(lib().ssd_load_weights(self.h, C.byref(w)))

    def w8_read(self, which: int, layer: int = 0):
        """ssd_w8_read: (codes uint8 [rows, cols], scales float32 [rows]) of one 8-bit matrix (which: 0 w_qkv, 1 w_o, 2 w_fc, 3 w_proj, 4 head)."""
        d, F, V = self.cfg["d_model"], self.cfg["d_ff"], self.cfg["vocab"]
        rows, cols = [(3 * d, d), (d, d), (F, d), (d, F), (V, d)][which]
        codes, scales = np.empty((rows, cols), dtype=np.uint8), np.empty(rows, dtype=np.float32)
        self._chk(lib().ssd_w8_read(self.h, which, layer, codes.ctypes.data, scales.ctypes.data))
        return codes, scales

    def new_kv(self) -> "KV":
        return KV(self)

    def verify_tree(self, tokens, parent_idx, kv: "KV", logits_out_ptr: int):
        """ssd_verify_tree.  ``logits_out_ptr``: device address of a [n, vocab] fp32 buffer."""
        tokens, parent_idx = _i32(tokens), _i32(parent_idx)
        assert len(tokens) == len(parent_idx)
        self._chk(lib().ssd_verify_tree(self.h, tokens.ctypes.data, parent_idx.ctypes.data, len(tokens), kv.h, _VP(logits_out_ptr)))

    def accept_tree(self, logits_ptr: int, draft_probs_ptr, tokens, parent_idx, mode: int = SSD_GREEDY, temperature: float = 1.0,
                    top_k: int = 0, rng: ssd_rng | None = None):
        """ssd_accept_tree.  Returns (path list, next_token); ``rng`` (an ssd_rng) is advanced in place."""
        tokens, parent_idx = _i32(tokens), _i32(parent_idx)
        n = len(tokens)
        samp = ssd_sampling(mode, temperature, top_k)
        rng = rng if rng is not None else ssd_rng(0, 0)
        path = np.zeros(max(n, 1), dtype=np.int32)
        n_path, nxt = C.c_int32(0), C.c_int32(-1)
        rc = lib().ssd_accept_tree(self.h, _VP(logits_ptr), _VP(draft_probs_ptr or 0), tokens.ctypes.data, parent_idx.ctypes.data, n,
                                   C.byref(samp), C.byref(rng), path.ctypes.data, C.byref(n_path), C.byref(nxt))
        self._chk(rc)
        return [int(v) for v in path[:n_path.value]], int(nxt.value)

    def accept_tree_sparse(self, logits_ptr: int, row_idx, row_val, tokens, parent_idx, mode: int = SSD_SAMPLING, temperature: float = 1.0,
                           top_k: int = 0, rng: ssd_rng | None = None):
        """ssd_accept_tree_sparse: proposal rows as [n, entries] index / value lists (index < 0 = unused slot)."""
        tokens, parent_idx = _i32(tokens), _i32(parent_idx)
        n = len(tokens)
        idx = np.ascontiguousarray(row_idx, dtype=np.int32).reshape(n, -1)
        val = np.ascontiguousarray(row_val, dtype=np.float32).reshape(n, -1)
        assert idx.shape == val.shape
        samp = ssd_sampling(mode, temperature, top_k)
        rng = rng if rng is not None else ssd_rng(0, 0)
        path = np.zeros(max(n, 1), dtype=np.int32)
        n_path, nxt = C.c_int32(0), C.c_int32(-1)
        rc = lib().ssd_accept_tree_sparse(self.h, _VP(logits_ptr), idx.ctypes.data, val.ctypes.data, idx.shape[1], tokens.ctypes.data,
                                          parent_idx.ctypes.data, n, C.byref(samp), C.byref(rng), path.ctypes.data, C.byref(n_path), C.byref(nxt))
        self._chk(rc)
        return [int(v) for v in path[:n_path.value]], int(nxt.value)

    def propose_children(self, logits_ptr: int, nodes, picks: int, mode: int = SSD_GREEDY, temperature: float = 1.0, top_k: int = 0,
                         rng: ssd_rng | None = None, rows_out_ptr: int = 0) -> np.ndarray:
        """ssd_propose_children.  Returns tokens int32 [len(nodes), picks]; the nodes' laws go to ``rows_out_ptr`` (device) if given."""
        nodes = _i32(nodes)
        samp = ssd_sampling(mode, temperature, top_k)
        rng = rng if rng is not None else ssd_rng(0, 0)
        out = np.zeros((len(nodes), max(picks, 1)), dtype=np.int32)
        self._chk(lib().ssd_propose_children(self.h, _VP(logits_ptr), nodes.ctypes.data, len(nodes), picks, C.byref(samp), C.byref(rng),
                                             _VP(rows_out_ptr or 0), out.ctypes.data))
        return out[:, :picks]

    def kv_commit(self, kv: "KV", path):
        path = _i32(path)
        self._chk(lib().ssd_kv_commit(self.h, kv.h, path.ctypes.data, len(path)))

    def kv_read(self, kv: "KV", layer: int, which: int, slot0: int, rows: int) -> np.ndarray:
        out = np.empty((rows, self.cfg["d_model"]), dtype=np.float32)
        self._chk(lib().ssd_kv_read(self.h, kv.h, layer, which, slot0, rows, out.ctypes.data))
        return out

    def set_tuning(self, knob: int, value: int):
        self._chk(lib().ssd_set_tuning(self.h, knob, value))

    def phase_trace(self) -> np.ndarray:
        out = np.zeros(4096, dtype=np.uint64)
        cnt = C.c_int32(0)
        self._chk(lib().ssd_get_phase_trace(self.h, out.ctypes.data, len(out), C.byref(cnt)))
        return out[:cnt.value].copy()

    def device_status(self) -> int:
        w = C.c_int32(0)
        self._chk(lib().ssd_last_device_status(self.h, C.byref(w)))
        return w.value

    def reset_device_status(self) -> None:
        self._chk(lib().ssd_reset_device_status(self.h))

    def debug_expire_wait(self, limit_us: int = 10) -> None:
        self._chk(lib().ssd_debug_expire_wait(self.h, int(limit_us)))

    def kernel_launches(self) -> int:
        c = C.c_int64(0)
        self._chk(lib().ssd_kernel_launches(self.h, C.byref(c)))
        return c.value


class KV:
    """ssd_kv: one sequence's cache."""

    def __init__(self, ctx: Context):
        self.ctx = ctx
        h = _VP()
        ctx._chk(lib().ssd_kv_create(ctx.h, C.byref(h)))
        self.h = h

    def close(self):
        if getattr(self, "h", None) and getattr(self.ctx, "h", None):
            lib().ssd_kv_destroy(self.h)
        self.h = None

    def __del__(self):
        self.close()

    def __len__(self):
        n = C.c_int32(0)
        self.ctx._chk(lib().ssd_kv_len(self.h, C.byref(n)))
        return n.value

    def reset(self):
        self.ctx._chk(lib().ssd_kv_reset(self.h))

    def rollback(self, n: int):
        self.ctx._chk(lib().ssd_kv_rollback(self.h, n))


class Trigram:
    """Handle of a Katz back-off trigram table on the device (argument marshalling only)."""

    def __init__(self, stream_tokens, vocab: int, device: int = 0, stream: int = 0):
        toks = np.ascontiguousarray(stream_tokens, dtype=np.int32)
        h = _VP()
        rc = lib().ssd_trigram_build(toks.ctypes.data, len(toks), int(vocab), int(device), _VP(stream), C.byref(h))
        if rc != SSD_OK:
            raise SsdError(rc)
        self.h, self.vocab = h, int(vocab)

    def lookup(self, contexts):
        """contexts: [m, 2] preceding token pairs -> (tokens int32 [m, 4], probabilities float32 [m, 4])."""
        ctx = np.ascontiguousarray(contexts, dtype=np.int32).reshape(-1, 2)
        tok = np.zeros((len(ctx), 4), dtype=np.int32)
        pr = np.zeros((len(ctx), 4), dtype=np.float32)
        rc = lib().ssd_trigram_lookup(self.h, ctx.ctypes.data, len(ctx), tok.ctypes.data, pr.ctypes.data)
        if rc != SSD_OK:
            raise SsdError(rc)
        return tok, pr

    def propose(self, prev1: int, root: int, parent_idx):
        par = np.ascontiguousarray(parent_idx, dtype=np.int32)
        tok = np.zeros(len(par), dtype=np.int32)
        pr = np.zeros(len(par), dtype=np.float32)
        rc = lib().ssd_trigram_propose(self.h, int(prev1), int(root), par.ctypes.data, len(par), tok.ctypes.data, pr.ctypes.data)
        if rc != SSD_OK:
            raise SsdError(rc)
        return tok, pr

    def contexts(self) -> int:
        c = C.c_int64(0)
        rc = lib().ssd_trigram_contexts(self.h, C.byref(c))
        if rc != SSD_OK:
            raise SsdError(rc)
        return c.value

    def close(self):
        if self.h:
            lib().ssd_trigram_destroy(self.h)
            self.h = None
