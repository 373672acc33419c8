"""Thin Python binding over liba3.so: argument marshalling only.

Every step of the fusion path runs inside the CUDA library; torch is used here for
device memory and streams.  Function names mirror the C ABI (include/a3.h).  The
library is loaded at first use and the import fails loudly when it has not been
built: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liba3.so")
_lib = None

A3_OK = 0
DEV_BAD_POSITION, DEV_NONFINITE_SCORE, DEV_WAIT_EXHAUSTED, DEV_UNSORTED_ROWS = 1, 2, 4, 8


class A3Error(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = _load()
        msg = lib.a3_status_string(status).decode()
        extra = f" (cudaError {lib.a3_last_cuda_error()})" if status == -4 else ""
        super().__init__(f"{where}: {msg}{extra} [{status}]")
        self.status = status


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("d_ff", C.c_int), ("rope_theta", C.c_double), ("rms_eps", C.c_float),
                ("rope_layout", C.c_int), ("max_positions", C.c_int)]


_W_FIELDS = ("attn_norm", "wq", "wk", "wv", "bq", "bk", "bv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _W_FIELDS]


class ChunkRef(C.Structure):
    _fields_ = [("k_src", C.c_void_p), ("v_src", C.c_void_p), ("src_layer_stride", C.c_uint64), ("len", C.c_int32),
                ("dst_offset", C.c_int32), ("delta", C.c_int32), ("token_step", C.c_int32)]


class Request(C.Structure):
    _fields_ = [("chunks", C.c_void_p), ("n_chunks", C.c_int32), ("max_chunk_len", C.c_int32), ("n_ctx", C.c_int32),
                ("n_question", C.c_int32), ("n_system", C.c_int32), ("select_layer", C.c_int32),
                ("n_recompute", C.c_int32), ("score_source", C.c_int32), ("selector", C.c_int32), ("reserved", C.c_int32), ("x0", C.c_void_p), ("k_fused", C.c_void_p),
                ("v_fused", C.c_void_p), ("layer_stride", C.c_uint64), ("forced_re", C.c_void_p),
                ("rows_out", C.c_void_p), ("scores_out", C.c_void_p), ("x_out", C.c_void_p),
                ("evict_capacity", C.c_int32), ("evict_pool", C.c_int32), ("k_evicted", C.c_void_p), ("v_evicted", C.c_void_p),
                ("evicted_layer_stride", C.c_uint64), ("kept_out", C.c_void_p)]


class HostIO(C.Structure):
    _fields_ = [("chunk_k", C.POINTER(C.c_void_p)), ("chunk_v", C.POINTER(C.c_void_p)), ("chunk_len", C.POINTER(C.c_int32)),
                ("x0", C.c_void_p), ("rows_out", C.c_void_p), ("x_out", C.c_void_p)]


# a3_option (include/a3.h)
(OPT_ATTN_SPLIT, OPT_ATTN_PAIR, OPT_ATTN_MAX_CTAS, OPT_SWIGLU_NARROW, OPT_SWIGLU_PAIR, OPT_RESIDUAL_T, OPT_GEMM_BN_RESIDUAL,
 OPT_GEMM_BN_SWIGLU, OPT_GEMM_BN_QKV, OPT_GEMM_STAGES_RESIDUAL, OPT_GEMM_STAGES_SWIGLU, OPT_GEMM_STAGES_QKV,
 OPT_SCORES_KERNEL, OPT_QKV_T, OPT_GEMM_TILING, OPT_COUNT) = range(16)

EXPORTS = ("a3_create", "a3_destroy", "a3_set_option", "a3_scores_workspace_bytes", "a3_swiglu_rows", "a3_layer_workspace_bytes", "a3_request_workspace_bytes", "a3_host_staging_bytes",
           "a3_recompute_count", "a3_rope_rerotate", "a3_query_scores", "a3_query_scores_static", "a3_topk_select", "a3_recompute_layer",
           "a3_scatter_kv", "a3_gather_rows", "a3_precompute_chunk", "a3_first_token_workspace_bytes", "a3_first_token",
           "a3_evict_count", "a3_evict_workspace_bytes", "a3_evict_layer", "a3_chunk_edge_rows", "a3_random_rows", "a3_fuse_request", "a3_fuse_batch", "a3_fuse_request_host",
           "a3_graph_capture", "a3_graph_launch", "a3_graph_kernel_count", "a3_graph_destroy",
           "a3_device_status", "a3_status_string", "a3_last_cuda_error", "a3_launch_count", "a3_profile_enable",
           "a3_profile_read", "a3_kernel_class_name")
K_CLASSES = 10


class ProfileEntry(C.Structure):
    _fields_ = [("launches", C.c_uint64), ("ms", C.c_double)]


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2511_17560_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, u64, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
    lib.a3_create.argtypes = [C.POINTER(vp), C.POINTER(ModelDesc), C.POINTER(LayerWeights)]
    lib.a3_destroy.argtypes = [vp]
    lib.a3_destroy.restype = None
    lib.a3_set_option.argtypes = [vp, i32, i32]
    lib.a3_swiglu_rows.argtypes = [vp, i32, vp, vp, i32, vp]
    for name in ("a3_layer_workspace_bytes", "a3_request_workspace_bytes", "a3_scores_workspace_bytes"):
        getattr(lib, name).argtypes = [vp, i32]
        getattr(lib, name).restype = sz
    lib.a3_host_staging_bytes.argtypes = [vp, i32, i32]
    lib.a3_host_staging_bytes.restype = sz
    lib.a3_recompute_count.argtypes = [C.c_double, i32, i32]
    lib.a3_rope_rerotate.argtypes = [vp, vp, i32, i32, vp, vp, u64, i32, i32, i32, vp]
    lib.a3_query_scores.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.a3_query_scores_static.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, vp, vp]
    lib.a3_topk_select.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    lib.a3_recompute_layer.argtypes = [vp, i32, vp, vp, i32, vp, vp, i32, vp, vp, sz, vp]
    lib.a3_scatter_kv.argtypes = [vp, vp, vp, vp, i32, vp, vp, i32, vp]
    lib.a3_gather_rows.argtypes = [vp, vp, i32, vp, i32, i32, vp, vp]
    lib.a3_precompute_chunk.argtypes = [vp, vp, i32, vp, vp, u64, vp, sz, vp]
    lib.a3_chunk_edge_rows.argtypes = [C.POINTER(C.c_int32), i32, i32, i32, C.POINTER(C.c_int32), i32]
    lib.a3_random_rows.argtypes = [u64, i32, i32, i32, C.POINTER(C.c_int32), i32]
    lib.a3_evict_count.argtypes = [i32, i32, i32, i32]
    lib.a3_evict_workspace_bytes.argtypes = [vp, i32]
    lib.a3_evict_workspace_bytes.restype = sz
    lib.a3_evict_layer.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    lib.a3_first_token_workspace_bytes.argtypes = [vp]
    lib.a3_first_token_workspace_bytes.restype = sz
    lib.a3_first_token.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, sz, vp]
    lib.a3_fuse_request.argtypes = [vp, C.POINTER(Request), vp, sz, vp]
    lib.a3_fuse_batch.argtypes = [vp, C.POINTER(Request), i32, vp, sz, vp]
    lib.a3_fuse_request_host.argtypes = [vp, C.POINTER(Request), C.POINTER(HostIO), vp, sz, vp, sz, vp]
    lib.a3_graph_capture.argtypes = [vp, C.POINTER(Request), vp, sz, vp, C.POINTER(vp)]
    lib.a3_graph_launch.argtypes = [vp, vp]
    lib.a3_graph_kernel_count.argtypes = [vp]
    lib.a3_graph_destroy.argtypes = [vp]
    lib.a3_graph_destroy.restype = None
    lib.a3_device_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    lib.a3_status_string.argtypes = [i32]
    lib.a3_status_string.restype = C.c_char_p
    lib.a3_last_cuda_error.argtypes = []
    lib.a3_launch_count.argtypes = [i32]
    lib.a3_launch_count.restype = u64
    lib.a3_profile_enable.argtypes = [vp, i32]
    lib.a3_profile_read.argtypes = [vp, C.POINTER(ProfileEntry), vp]
    lib.a3_kernel_class_name.argtypes = [i32]
    lib.a3_kernel_class_name.restype = C.c_char_p
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != A3_OK:
        raise A3Error(status, where)


def recompute_count(ratio: float, n: int, n_candidates: int) -> int:
    return int(_load().a3_recompute_count(float(ratio), int(n), int(n_candidates)))


def chunk_edge_rows(chunk_lens: Sequence[int], m: int, n_system: int = 0) -> np.ndarray:
    """Slots of the first/last m tokens of every chunk (ascending), for use as forced_re."""
    lens = (C.c_int32 * max(1, len(chunk_lens)))(*[int(t) for t in chunk_lens])
    count = int(_load().a3_chunk_edge_rows(lens, len(chunk_lens), int(m), int(n_system), None, 0))
    out = (C.c_int32 * max(1, count))()
    _load().a3_chunk_edge_rows(lens, len(chunk_lens), int(m), int(n_system), out, count)
    return np.frombuffer(out, dtype=np.int32, count=count).copy()


def random_rows(seed: int, cand_begin: int, cand_end: int, k: int) -> np.ndarray:
    """k distinct candidate slots drawn uniformly at random (ascending), for use as forced_re."""
    k = max(0, min(int(k), cand_end - cand_begin))
    out = (C.c_int32 * max(1, k))()
    count = int(_load().a3_random_rows(int(seed), int(cand_begin), int(cand_end), k, out, k))
    return np.frombuffer(out, dtype=np.int32, count=count).copy()


def evict_count(capacity: int, n_system: int, n_ctx: int, n_question: int) -> int:
    return int(_load().a3_evict_count(int(capacity), int(n_system), int(n_ctx), int(n_question)))


class RequestGraph:
    """A request captured by a3_graph_capture: launch() replays it on the current stream."""

    def __init__(self, handle, req, ws):
        self._g, self._req, self._ws = handle, req, ws

    def launch(self):
        _check(_load().a3_graph_launch(self._g, _stream()), "a3_graph_launch")

    @property
    def kernels(self) -> int:
        return int(_load().a3_graph_kernel_count(self._g))

    def close(self):
        if self._g:
            _load().a3_graph_destroy(self._g)
            self._g = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def launch_count(reset: bool = False) -> int:
    return int(_load().a3_launch_count(1 if reset else 0))


def chunk_table(chunk_k: Sequence[torch.Tensor], chunk_v: Sequence[torch.Tensor], offsets: Sequence[int],
                deltas: Optional[Sequence[int]] = None, device=None, token_step: int = 0) -> torch.Tensor:
    """Device array of a3_chunk_ref for chunk caches shaped [L][T][Hkv][D] (bf16, contiguous).
    token_step: 0 for keys stored at local positions, 1 for keys stored without positional embedding,
    -1 (with deltas of 0) to strip the local positions."""
    arr = (ChunkRef * max(1, len(chunk_k)))()
    for c, (k, v) in enumerate(zip(chunk_k, chunk_v)):
        assert k.dtype == torch.bfloat16 and k.is_contiguous() and v.is_contiguous() and k.shape == v.shape
        arr[c].k_src, arr[c].v_src = k.data_ptr(), v.data_ptr()
        arr[c].src_layer_stride = k.stride(0) * 2
        arr[c].len = k.shape[1]
        arr[c].dst_offset = int(offsets[c])
        arr[c].delta = int(offsets[c] if deltas is None else deltas[c])
        arr[c].token_step = int(token_step)
    raw = np.frombuffer(bytes(arr), dtype=np.uint8).copy()
    dev = device if device is not None else (chunk_k[0].device if len(chunk_k) else "cuda")
    return torch.from_numpy(raw).to(dev)


class A3:
    """Owns an a3_handle; keeps the weight tensors alive (the library only borrows their pointers)."""

    def __init__(self, shape, weights: List[Dict[str, torch.Tensor]], max_positions: int):
        lib = _load()
        self.shape = shape
        self._weights = weights
        self.desc = ModelDesc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                              shape.d_ff, float(shape.rope_theta), float(shape.rms_eps), int(shape.rope_layout),
                              int(max_positions))
        arr = (LayerWeights * shape.n_layers)()
        for l, w in enumerate(weights):
            for name in _W_FIELDS:
                t = w.get(name)
                if t is not None:
                    assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous(), name
                setattr(arr[l], name, _ptr(t))
        self._h = C.c_void_p()
        _check(lib.a3_create(C.byref(self._h), C.byref(self.desc), arr), "a3_create")
        self.device = weights[0]["wq"].device
        self._ws: Optional[torch.Tensor] = None

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            _load().a3_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- workspace
    def layer_workspace_bytes(self, max_rows: int) -> int:
        return int(_load().a3_layer_workspace_bytes(self._h, int(max_rows)))

    def request_workspace_bytes(self, n: int) -> int:
        return int(_load().a3_request_workspace_bytes(self._h, int(n)))

    def host_staging_bytes(self, n_ctx: int, n: int) -> int:
        return int(_load().a3_host_staging_bytes(self._h, int(n_ctx), int(n)))

    def workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(int(nbytes) + 256, dtype=torch.uint8, device=self.device)
        return self._ws

    # ---- the steps (names as in the C ABI)
    def set_option(self, option: int, value: int):
        """a3_set_option: pins a kernel variant on this handle (cross-checks and measurements)."""
        _check(_load().a3_set_option(self._h, int(option), int(value)), "a3_set_option")

    def rope_rerotate(self, chunks: torch.Tensor, n_chunks: int, max_chunk_len: int, k_fused: torch.Tensor,
                      v_fused: torch.Tensor, layer_begin: int = 0, layer_end: Optional[int] = None, kv_len: Optional[int] = None):
        """kv_len: slots of a fused layer (default: the tensor's second dimension)."""
        layer_end = self.shape.n_layers if layer_end is None else layer_end
        stride = k_fused.stride(0) * 2
        kv_len = k_fused.shape[1] if kv_len is None else kv_len
        _check(_load().a3_rope_rerotate(self._h, _ptr(chunks), n_chunks, max_chunk_len, _ptr(k_fused), _ptr(v_fused),
                                        stride, kv_len, layer_begin, layer_end, _stream()), "a3_rope_rerotate")

    def swiglu_rows(self, layer: int, x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if out is None:
            out = torch.empty((x.shape[0], self.shape.d_ff), dtype=torch.bfloat16, device=x.device)
        _check(_load().a3_swiglu_rows(self._h, layer, _ptr(x), _ptr(out), x.shape[0], _stream()), "a3_swiglu_rows")
        return out

    def query_scores(self, q_rows, q_pos, k_layer, cand_begin, cand_end, lse=None, scores=None):
        nq, kv_len = q_rows.shape[0], k_layer.shape[0]
        if scores is None:
            scores = torch.empty(kv_len, dtype=torch.float32, device=k_layer.device)
        ws = self.workspace(int(_load().a3_scores_workspace_bytes(self._h, nq)))
        _check(_load().a3_query_scores(self._h, _ptr(q_rows), _ptr(q_pos), nq, _ptr(k_layer), kv_len, cand_begin,
                                       cand_end, _ptr(lse), _ptr(scores), _ptr(ws), ws.numel(), _stream()),
               "a3_query_scores")
        return scores

    def query_scores_static(self, q_rows, q_pos, k_layer, cand_begin, cand_end, scores=None):
        """a3_query_scores for callers that cannot allocate: no workspace, scratch inside the library image.

        Limited to q_rows.shape[0] * n_q_heads <= 65536; calls that may overlap on the GPU must be ordered by the
        caller because they share that scratch.  Only `scores` (an output) is created here when not supplied.
        """
        nq, kv_len = q_rows.shape[0], k_layer.shape[0]
        if scores is None:
            scores = torch.empty(kv_len, dtype=torch.float32, device=k_layer.device)
        _check(_load().a3_query_scores_static(self._h, _ptr(q_rows), _ptr(q_pos), nq, _ptr(k_layer), kv_len, cand_begin,
                                              cand_end, _ptr(scores), _stream()), "a3_query_scores_static")
        return scores

    def topk_select(self, scores, cand_begin, cand_end, k, idx_out=None):
        kk = max(0, min(k, cand_end - cand_begin))
        if idx_out is None:
            idx_out = torch.empty(kk, dtype=torch.int32, device=scores.device)
        _check(_load().a3_topk_select(self._h, _ptr(scores), cand_begin, cand_end, k, _ptr(idx_out), _stream()),
               "a3_topk_select")
        return idx_out

    def recompute_layer(self, layer, x_rows, pos, k_layer, v_layer, lse_out=None):
        M, kv_len = x_rows.shape[0], k_layer.shape[0]
        ws = self.workspace(self.layer_workspace_bytes(max(M, 1)))
        _check(_load().a3_recompute_layer(self._h, layer, _ptr(x_rows), _ptr(pos), M, _ptr(k_layer), _ptr(v_layer),
                                          kv_len, _ptr(lse_out), _ptr(ws), ws.numel(), _stream()), "a3_recompute_layer")
        return x_rows

    def scatter_kv(self, k_rows, v_rows, slots, k_layer, v_layer):
        _check(_load().a3_scatter_kv(self._h, _ptr(k_rows), _ptr(v_rows), _ptr(slots), k_rows.shape[0], _ptr(k_layer),
                                     _ptr(v_layer), k_layer.shape[0], _stream()), "a3_scatter_kv")

    def gather_rows(self, src, rows, dst=None):
        M, width = rows.shape[0], src.shape[1]
        if dst is None:
            dst = torch.empty((M, width), dtype=src.dtype, device=src.device)
        _check(_load().a3_gather_rows(self._h, _ptr(src), src.shape[0], _ptr(rows), M, width, _ptr(dst), _stream()),
               "a3_gather_rows")
        return dst

    def precompute_chunk(self, x_chunk, k_chunk, v_chunk):
        """Eq. 1 for one chunk: x_chunk [T][d] in/out, k_chunk/v_chunk [L][T][Hkv][D] filled."""
        T = x_chunk.shape[0]
        ws = self.workspace(self.request_workspace_bytes(max(T, 1)))
        _check(_load().a3_precompute_chunk(self._h, _ptr(x_chunk), T, _ptr(k_chunk), _ptr(v_chunk), k_chunk.stride(0) * 2,
                                           _ptr(ws), ws.numel(), _stream()), "a3_precompute_chunk")
        return x_chunk

    def evict_layer(self, q_window, q_pos, lse, k_layer, v_layer, n_system, n_ctx, capacity, pool=1):
        """`ex` for one layer; returns (k_out, v_out, kept) with C' = n_system + k + nq entries per head."""
        nq = q_pos.shape[0]
        kv_len = k_layer.shape[0]
        Cp = n_system + evict_count(capacity, n_system, n_ctx, nq) + nq
        Hkv, D = self.shape.n_kv_heads, self.shape.head_dim
        k_out = torch.zeros((Cp, Hkv, D), dtype=torch.bfloat16, device=k_layer.device)
        v_out = torch.zeros_like(k_out)
        kept = torch.full((Hkv, Cp), -1, dtype=torch.int32, device=k_layer.device)
        ws = self.workspace(int(_load().a3_evict_workspace_bytes(self._h, kv_len)))
        _check(_load().a3_evict_layer(self._h, _ptr(q_window), _ptr(q_pos), nq, _ptr(lse), _ptr(k_layer), _ptr(v_layer), kv_len,
                                      n_system, n_ctx, capacity, pool, _ptr(k_out), _ptr(v_out), _ptr(kept), _ptr(ws), ws.numel(),
                                      _stream()), "a3_evict_layer")
        return k_out, v_out, kept

    def first_token(self, x_row, final_norm, lm_head, want_logits=True):
        """Final norm + vocabulary projection + greedy choice for one hidden row [d]; returns (logits or None, token)."""
        vocab = lm_head.shape[0]
        dev = lm_head.device
        logits = torch.empty(vocab, dtype=torch.float32, device=dev) if want_logits else None
        token = torch.empty(1, dtype=torch.int32, device=dev)
        ws = self.workspace(int(_load().a3_first_token_workspace_bytes(self._h)))
        _check(_load().a3_first_token(self._h, _ptr(x_row), _ptr(final_norm), _ptr(lm_head), vocab, _ptr(logits), _ptr(token),
                                      _ptr(ws), ws.numel(), _stream()), "a3_first_token")
        return logits, token

    def make_request(self, chunks, n_chunks, max_chunk_len, n_ctx, n_question, x0, k_fused, v_fused, ratio=0.15,
                     select_layer=1, n_system=0, forced_re=None, n_recompute=None, score_source=0, evict_capacity=0,
                     evict_pool=1, selector=0):
        """Allocates the outputs and fills an a3_request; returns (Request, dict of output tensors)."""
        n = n_ctx + n_question
        p = recompute_count(ratio, n, n_ctx - n_system) if n_recompute is None else n_recompute
        if forced_re is not None:
            p = int(forced_re.shape[0])
        dev = k_fused.device
        out = dict(rows=torch.empty(p + n_question, dtype=torch.int32, device=dev),
                   scores=torch.empty(n, dtype=torch.float32, device=dev),
                   x=torch.empty((p + n_question, self.shape.d_model), dtype=torch.bfloat16, device=dev),
                   p=p)
        r = Request()
        r.chunks, r.n_chunks, r.max_chunk_len = _ptr(chunks), n_chunks, max_chunk_len
        r.n_ctx, r.n_question, r.n_system = n_ctx, n_question, n_system
        r.select_layer, r.n_recompute, r.score_source = select_layer, p, int(score_source)
        r.selector = int(selector)
        r.x0, r.k_fused, r.v_fused = _ptr(x0), _ptr(k_fused), _ptr(v_fused)
        r.layer_stride = k_fused.stride(0) * 2
        r.forced_re = _ptr(forced_re)
        r.rows_out, r.scores_out, r.x_out = _ptr(out["rows"]), _ptr(out["scores"]), _ptr(out["x"])
        if evict_capacity > 0:
            L, Hkv, D = self.shape.n_layers, self.shape.n_kv_heads, self.shape.head_dim
            Cp = n_system + evict_count(evict_capacity, n_system, n_ctx, n_question) + n_question
            out["k_evicted"] = torch.zeros((L, Cp, Hkv, D), dtype=torch.bfloat16, device=dev)
            out["v_evicted"] = torch.zeros_like(out["k_evicted"])
            out["kept"] = torch.full((L, Hkv, Cp), -1, dtype=torch.int32, device=dev)
            r.evict_capacity, r.evict_pool = int(evict_capacity), int(evict_pool)
            r.k_evicted, r.v_evicted, r.kept_out = _ptr(out["k_evicted"]), _ptr(out["v_evicted"]), _ptr(out["kept"])
            r.evicted_layer_stride = out["k_evicted"].stride(0) * 2
        out["_keep"] = (chunks, x0, k_fused, v_fused, forced_re)
        return r, out

    def fuse_request(self, req: Request):
        n = req.n_ctx + req.n_question
        ws = self.workspace(self.request_workspace_bytes(n))
        _check(_load().a3_fuse_request(self._h, C.byref(req), _ptr(ws), ws.numel(), _stream()), "a3_fuse_request")

    def graph_capture(self, req: Request) -> "RequestGraph":
        """a3_graph_capture on the current stream (not the default stream); the graph keeps `req` and a workspace of
        its own alive."""
        n = req.n_ctx + req.n_question
        ws = torch.empty(int(self.request_workspace_bytes(n)) + 256, dtype=torch.uint8, device=self.device)
        g = C.c_void_p()
        _check(_load().a3_graph_capture(self._h, C.byref(req), _ptr(ws), ws.numel(), _stream(), C.byref(g)), "a3_graph_capture")
        return RequestGraph(g, req, ws)

    def fuse_batch(self, reqs: Sequence[Request]):
        arr = (Request * len(reqs))(*reqs)
        n = max(r.n_ctx + r.n_question for r in reqs)
        ws = self.workspace(self.request_workspace_bytes(n))
        _check(_load().a3_fuse_batch(self._h, arr, len(reqs), _ptr(ws), ws.numel(), _stream()), "a3_fuse_batch")

    def fuse_request_host(self, req: Request, chunk_k: Sequence[torch.Tensor], chunk_v: Sequence[torch.Tensor],
                          x0: torch.Tensor, rows_out: torch.Tensor, x_out: torch.Tensor, staging: torch.Tensor):
        """Chunk caches, embeddings and the two result buffers are HOST tensors (pinned recommended)."""
        nc = len(chunk_k)
        ks = (C.c_void_p * max(nc, 1))(*[t.data_ptr() for t in chunk_k])
        vs = (C.c_void_p * max(nc, 1))(*[t.data_ptr() for t in chunk_v])
        ls = (C.c_int32 * max(nc, 1))(*[int(t.shape[1]) for t in chunk_k])
        io = HostIO(ks, vs, ls, x0.data_ptr(), rows_out.data_ptr(), x_out.data_ptr())
        n = req.n_ctx + req.n_question
        ws = self.workspace(self.request_workspace_bytes(n))
        _check(_load().a3_fuse_request_host(self._h, C.byref(req), C.byref(io), _ptr(staging), staging.numel(),
                                            _ptr(ws), ws.numel(), _stream()), "a3_fuse_request_host")

    def profile_enable(self, max_records: int):
        _check(_load().a3_profile_enable(self._h, int(max_records)), "a3_profile_enable")

    def profile_read(self) -> Dict[str, Dict[str, float]]:
        """Per kernel class: launches and summed device milliseconds since the last read (waits for the stream)."""
        lib = _load()
        arr = (ProfileEntry * K_CLASSES)()
        _check(lib.a3_profile_read(self._h, arr, _stream()), "a3_profile_read")
        return {lib.a3_kernel_class_name(k).decode(): dict(launches=int(arr[k].launches), ms=float(arr[k].ms))
                for k in range(K_CLASSES)}

    def device_status(self) -> int:
        bits = C.c_uint32(0)
        _check(_load().a3_device_status(self._h, C.byref(bits), _stream()), "a3_device_status")
        return int(bits.value)
