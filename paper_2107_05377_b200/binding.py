"""ctypes binding of the C-ABI library (``include/mt_bert.h``), same names.

Argument marshalling only: every step of the forward pass runs in the CUDA
kernels of ``libmt_bert.so``.  PyTorch appears only as the owner of device
memory and streams in the ``MTModel`` convenience wrapper.  There is no
fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libmt_bert.so")

MT_OK = 0
ERRORS = {0: "OK", -1: "INVALID_ARG", -2: "SHAPE", -3: "NOT_BOUND", -4: "NOT_LOADED", -5: "BLOB_MISMATCH",
          -6: "CUDA", -7: "UNSUPPORTED", -8: "DEVICE_FLAG"}
FLAG_BAD_TOKEN, FLAG_BAD_SEGMENT, FLAG_BAD_LENGTH, FLAG_WAIT_TIMEOUT = 1, 2, 4, 8
KERNEL_CLASSES = ("embed", "qkv", "attention", "attn_out", "ln1", "ffn_up", "ffn_down", "ln2", "head", "quant")


class TrunkConfig(C.Structure):
    _fields_ = [("vocab_size", C.c_int32), ("max_position", C.c_int32), ("type_vocab", C.c_int32),
                ("hidden", C.c_int32), ("heads", C.c_int32), ("ffn", C.c_int32), ("trunk_layers", C.c_int32),
                ("ln_eps", C.c_float), ("activation", C.c_int32)]


class TaskConfig(C.Structure):
    _fields_ = [("fork_depth", C.c_int32), ("branch_layers", C.c_int32), ("num_classes", C.c_int32),
                ("head_kind", C.c_int32)]


# name -> (restype, argtypes); the list is also what the symbol-export test checks.
_P, _I32, _U64, _SZ = C.c_void_p, C.c_int32, C.c_uint64, C.c_size_t
SIGNATURES = {
    "mt_create": (C.c_int, [C.POINTER(TrunkConfig), C.POINTER(TaskConfig), _I32, _I32, _I32, C.POINTER(_P)]),
    "mt_destroy": (None, [_P]),
    "mt_weights_bytes": (_SZ, [_P]),
    "mt_workspace_bytes": (_SZ, [_P]),
    "mt_bind_memory": (C.c_int, [_P, _P, _SZ, _P, _SZ]),
    "mt_blob_bytes": (_SZ, [_P]),
    "mt_task_blob_bytes": (_SZ, [_P, _I32]),
    "mt_load_weights": (C.c_int, [_P, _P, _SZ, _P]),
    "mt_adopt_weights": (C.c_int, [_P, _P]),
    "mt_load_task_weights": (C.c_int, [_P, _I32, _P, _SZ, _P]),
    "mt_forward": (C.c_int, [_P, _P, _P, _P, _U64, _I32, _I32, _P, _P]),
    "mt_forward_events": (C.c_int, [_P, _P, _P, _P, _U64, _I32, _I32, _P, C.POINTER(_P), _P]),
    "mt_forward_tokens": (C.c_int, [_P, _P, _P, _P, _U64, _I32, _I32, _P, _P, C.POINTER(_P), _P]),
    "mt_forward_host": (C.c_int, [_P, _P, _P, _P, _U64, _I32, _I32, _P, _P]),
    "mt_forward_host_async": (C.c_int, [_P, _P, _P, _P, _U64, _I32, _I32, _P, _P]),
    "mt_poll_status": (C.c_int, [_P, _P, C.POINTER(C.c_uint32)]),
    "mt_plan_summary": (C.c_int, [_P, _U64, C.POINTER(_I32), C.POINTER(_I32), C.POINTER(_I32), C.POINTER(_I32)]),
    "mt_plan_launches": (C.c_int, [_P, _U64, C.POINTER(_I32)]),
    "mt_plan_cache_size": (C.c_int, [_P]),
    "mt_set_option": (C.c_int, [_P, C.c_char_p, C.c_int64]),
    "mt_debug_copy_hidden": (C.c_int, [_P, _I32, _I32, _P, _P]),
    "mt_profile_read": (C.c_int, [_P, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "mt_last_error_string": (C.c_char_p, [_P]),
    "mt_kernel_linear_force_block_n": (None, [C.c_int32]),
    "mt_kernel_linear": (C.c_int, [_P, _P, _P, _P, _P, _I32, _I32, _I32, _I32, _I32, _P, _P]),
    "mt_kernel_quantize_rows": (C.c_int, [_P, _P, _P, _I32, _I32, _P]),
    "mt_kernel_linear_fp8": (C.c_int, [_P, _P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _I32, _P, _P]),
    "mt_kernel_linear_layernorm": (C.c_int, [_P, _P, _P, _P, _P, _P, _P, _P, _I32, _I32, _I32, C.c_float, _P, _P]),
    "mt_kernel_linear_layernorm_tiles": (C.c_int, [_P, _P, _P, _P, _P, _P, _P, _P, _I32, _I32, _I32, C.c_float, _I32, _P, _P]),
    "mt_kernel_attention": (C.c_int, [_P, _P, _P, _I32, _I32, _I32, _I32, _P, _P]),
    "mt_kernel_layernorm": (C.c_int, [_P, _P, _P, _P, _P, _I32, _I32, C.c_float, _P]),
    "mt_kernel_linear_partial": (C.c_int, [_P, _P, _P, _I32, _I32, _I32, _I32, _I32, _P, _P]),
    "mt_debug_wait_probe": (C.c_int, [C.c_uint64, _I32, _P, _P, _P, _P]),
    "mt_kernel_layernorm_partial": (C.c_int, [_P, _I32, _I32, _P, _P, _P, _P, _P, _P, _I32, _I32, C.c_float, _P]),
    "mt_kernel_embed": (C.c_int, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _I32, _I32, C.c_float, _P,
                                  _P]),
    "mt_kernel_pooler_head": (C.c_int, [_P, _P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _I32, _I32, _I32, _P]),
    "mt_kernel_pooler_head_static": (C.c_int, [_P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _I32, _I32, _I32, _P]),
}

_lib = None


def lib() -> C.CDLL:
    """Loads libmt_bert.so (built by ``python -m paper_2107_05377_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2107_05377_b200.build` "
                               "(there is no fallback path)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


class MTError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        super().__init__(f"{where}: {ERRORS.get(code, code)} {detail}".strip())
        self.code = code


def _check(code: int, where: str, model=None) -> None:
    if code != MT_OK:
        detail = lib().mt_last_error_string(model).decode() if model else ""
        raise MTError(code, where, detail)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def torch_stream_for_init():
    import torch
    return torch.cuda.current_stream()


def _stream(stream=None) -> int:
    import torch
    return (stream or torch.cuda.current_stream()).cuda_stream


# ---------------------------------------------------------------------------
# single steps (device tensors in, device tensors out)
# ---------------------------------------------------------------------------

def mt_kernel_linear(x, w, bias, residual, y, epilogue: int, status=None, stream=None, cta_pair: bool = False) -> None:
    M, K = x.shape
    N = w.shape[0]
    _check(lib().mt_kernel_linear(_ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(y), M, N, K, epilogue,
                                  1 if cta_pair else 0, _ptr(status), _stream(stream)), "mt_kernel_linear")


def mt_kernel_quantize_rows(x, q, scale, stream=None) -> None:
    rows, cols = x.shape
    _check(lib().mt_kernel_quantize_rows(_ptr(x), _ptr(q), _ptr(scale), rows, cols, _stream(stream)),
           "mt_kernel_quantize_rows")


def mt_kernel_linear_fp8(xq, scale_x, wq, scale_w, bias, residual, y, epilogue: int, status=None, stream=None) -> None:
    M, K = xq.shape
    N = wq.shape[0]
    _check(lib().mt_kernel_linear_fp8(_ptr(xq), _ptr(scale_x), _ptr(wq), _ptr(scale_w), _ptr(bias), _ptr(residual),
                                      _ptr(y), M, N, K, epilogue, _ptr(status), _stream(stream)), "mt_kernel_linear_fp8")


def mt_kernel_linear_layernorm(x, w, bias, residual, gamma, beta, y, y_f32, eps: float, status=None, stream=None,
                               tile_cols: int = 128) -> None:
    M, K = x.shape
    N = w.shape[0]
    _check(lib().mt_kernel_linear_layernorm_tiles(_ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(gamma), _ptr(beta),
                                                  _ptr(y), _ptr(y_f32), M, N, K, eps, tile_cols, _ptr(status),
                                                  _stream(stream)), "mt_kernel_linear_layernorm_tiles")


def mt_kernel_attention(qkv, lengths, ctx, batch: int, seq: int, heads: int, stream=None,
                        tensor_memory: bool = False, status=None) -> None:
    _check(lib().mt_kernel_attention(_ptr(qkv), _ptr(lengths), _ptr(ctx), batch, seq, heads,
                                     1 if tensor_memory else 0, _ptr(status), _stream(stream)), "mt_kernel_attention")


def mt_kernel_layernorm(x, gamma, beta, y, eps: float, y_f32=None, stream=None) -> None:
    rows, hidden = x.shape
    _check(lib().mt_kernel_layernorm(_ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), _ptr(y_f32), rows, hidden, eps,
                                     _stream(stream)), "mt_kernel_layernorm")


def mt_debug_wait_probe(limit_ns: int, arrive: bool, status, waited_ns, ok, stream=None) -> None:
    """The kernels' bounded mbarrier wait on a barrier that nothing completes (arrive False) or that is complete."""
    _check(lib().mt_debug_wait_probe(int(limit_ns), 1 if arrive else 0, _ptr(status), _ptr(waited_ns), _ptr(ok),
                                     _stream(stream)), "mt_debug_wait_probe")


def mt_kernel_linear_partial(x, w, part, k_splits: int, split_pitch: int, status=None, stream=None) -> None:
    """part[s * split_pitch + i, :] = x[i, range s of K] . w[:, range s of K]^T (fp32, no bias)."""
    M, K = x.shape
    N = w.shape[0]
    _check(lib().mt_kernel_linear_partial(_ptr(x), _ptr(w), _ptr(part), M, N, K, k_splits, split_pitch, _ptr(status),
                                          _stream(stream)), "mt_kernel_linear_partial")


def mt_kernel_layernorm_partial(part, n_parts: int, part_pitch: int, residual, bias, gamma, beta, y, eps: float,
                                y_f32=None, stream=None) -> None:
    """y = LayerNorm(residual + ((part_0 + part_1 + ...) + bias))."""
    rows, hidden = residual.shape
    _check(lib().mt_kernel_layernorm_partial(_ptr(part), n_parts, part_pitch, _ptr(residual), _ptr(bias), _ptr(gamma),
                                             _ptr(beta), _ptr(y), _ptr(y_f32), rows, hidden, eps, _stream(stream)),
           "mt_kernel_layernorm_partial")


def mt_kernel_embed(token_ids, segment_ids, lengths, word, pos, type_, gamma, beta, h0, eps: float, h0_f32=None,
                    status=None, stream=None) -> None:
    batch, seq = token_ids.shape
    _check(lib().mt_kernel_embed(_ptr(token_ids), _ptr(segment_ids), _ptr(lengths), _ptr(word), _ptr(pos), _ptr(type_),
                                 _ptr(gamma), _ptr(beta), _ptr(h0), _ptr(h0_f32), batch, seq, word.shape[1], word.shape[0],
                                 type_.shape[0], eps, _ptr(status), _stream(stream)), "mt_kernel_embed")


def mt_kernel_pooler_head(hidden, pool_w, pool_b, cls_w, cls_b, pooled_scratch, logits, batch: int, seq: int,
                          col0: int = 0, stream=None) -> None:
    _check(lib().mt_kernel_pooler_head(_ptr(hidden), _ptr(pool_w), _ptr(pool_b), _ptr(cls_w), _ptr(cls_b),
                                       _ptr(pooled_scratch), _ptr(logits),
                                       batch, seq, pool_w.shape[0], cls_w.shape[0], logits.shape[1], col0,
                                       _stream(stream)), "mt_kernel_pooler_head")


STATIC_POOLER_MAX_FLOATS = 256 * 1024


def mt_kernel_pooler_head_static(hidden, pool_w, pool_b, cls_w, cls_b, logits, batch: int, seq: int, col0: int = 0,
                                 stream=None) -> None:
    """Pooler + head without a scratch argument, for callers that cannot allocate device memory:
    the features between the two launches go through a 1 MiB array built into the library
    (batch * hidden <= STATIC_POOLER_MAX_FLOATS).  Calls sharing a device must not overlap."""
    _check(lib().mt_kernel_pooler_head_static(_ptr(hidden), _ptr(pool_w), _ptr(pool_b), _ptr(cls_w), _ptr(cls_b),
                                              _ptr(logits), batch, seq, pool_w.shape[0], cls_w.shape[0],
                                              logits.shape[1], col0, _stream(stream)), "mt_kernel_pooler_head_static")


# ---------------------------------------------------------------------------
# the model
# ---------------------------------------------------------------------------

class MTModel:
    """mt_create + mt_bind_memory + mt_load_weights + mt_forward around torch-owned memory."""

    def __init__(self, cfg, max_batch: int, max_seq: int, max_groups: Optional[int] = None,
                 debug_capture: bool = False, device: str = "cuda:0", bind: bool = True, share_weights_with=None,
                 fp8_gemm: bool = False):
        """``share_weights_with``: another MTModel of the same configuration whose weights arena this one
        uses too (mt_adopt_weights) - a second batch in flight needs a workspace of its own, not a second
        copy of the weights."""
        self.cfg = cfg
        self.max_batch, self.max_seq = max_batch, max_seq
        self.handle = _P()
        trunk = TrunkConfig(cfg.vocab_size, cfg.max_position, cfg.type_vocab, cfg.hidden, cfg.heads, cfg.ffn,
                            cfg.trunk_layers, cfg.ln_eps, 0)
        tasks = (TaskConfig * cfg.n_tasks)(*[TaskConfig(t.fork_depth, t.branch_layers, t.num_classes, 1 if t.token_level else 0)
                                             for t in cfg.tasks])
        _check(lib().mt_create(C.byref(trunk), tasks, cfg.n_tasks, max_batch, max_seq, C.byref(self.handle)),
               "mt_create")
        if max_groups is not None:
            self.set_option("max_groups", max_groups)
        if debug_capture:
            self.set_option("debug_capture", 1)
        if fp8_gemm:
            self.set_option("fp8_gemm", 1)
        self.c_total = cfg.total_classes
        self.weights = self.workspace = None
        self._shared_from = share_weights_with
        if bind:
            self.bind(device)
            if share_weights_with is not None:
                _check(lib().mt_adopt_weights(self.handle, share_weights_with.handle), "mt_adopt_weights", self.handle)

    # -- host-only ----------------------------------------------------------
    def set_option(self, key: str, value: int) -> None:
        _check(lib().mt_set_option(self.handle, key.encode(), value), "mt_set_option", self.handle)

    def weights_bytes(self) -> int:
        return lib().mt_weights_bytes(self.handle)

    def workspace_bytes(self) -> int:
        return lib().mt_workspace_bytes(self.handle)

    def blob_bytes(self) -> int:
        return lib().mt_blob_bytes(self.handle)

    def task_blob_bytes(self, task: int) -> int:
        return lib().mt_task_blob_bytes(self.handle, task)

    def plan_summary(self, task_mask: int):
        n_layers, n_waves, depth = _I32(), _I32(), _I32()
        cap = self.cfg.trunk_layers + max(t.branch_layers for t in self.cfg.tasks) + 1
        groups = (_I32 * cap)()
        _check(lib().mt_plan_summary(self.handle, task_mask, C.byref(n_layers), C.byref(n_waves), C.byref(depth),
                                     groups), "mt_plan_summary", self.handle)
        return {"layers": n_layers.value, "waves": n_waves.value, "trunk_depth": depth.value,
                "groups_per_wave": list(groups[:n_waves.value])}

    def plan_launches(self, task_mask: int) -> int:
        n = _I32()
        _check(lib().mt_plan_launches(self.handle, task_mask, C.byref(n)), "mt_plan_launches", self.handle)
        return n.value

    def plan_cache_size(self) -> int:
        return lib().mt_plan_cache_size(self.handle)

    # -- device -------------------------------------------------------------
    def bind(self, device: str = "cuda:0") -> None:
        import torch
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.weights = self._shared_from.weights if self._shared_from is not None else \
            torch.empty(self.weights_bytes(), dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(self.workspace_bytes(), dtype=torch.uint8, device=self.device)
        _check(lib().mt_bind_memory(self.handle, self.weights.data_ptr(), self.weights.numel(),
                                    self.workspace.data_ptr(), self.workspace.numel()), "mt_bind_memory", self.handle)

    def load_weights(self, blob, stream=None) -> None:
        """``blob``: numpy uint8 array or torch CPU uint8 tensor (pinned for an asynchronous copy)."""
        import torch
        t = blob if isinstance(blob, torch.Tensor) else torch.from_numpy(blob)
        _check(lib().mt_load_weights(self.handle, t.data_ptr(), t.numel(), _stream(stream)), "mt_load_weights",
               self.handle)
        torch.cuda.current_stream().synchronize()

    def load_task_weights(self, task: int, blob, stream=None) -> None:
        import torch
        t = blob if isinstance(blob, torch.Tensor) else torch.from_numpy(blob)
        _check(lib().mt_load_task_weights(self.handle, task, t.data_ptr(), t.numel(), _stream(stream)),
               "mt_load_task_weights", self.handle)
        torch.cuda.current_stream().synchronize()

    def full_mask(self) -> int:
        return (1 << self.cfg.n_tasks) - 1

    def forward(self, token_ids, segment_ids, lengths, logits, task_mask: Optional[int] = None, stream=None) -> None:
        """Device int32 tensors in, fp32 ``logits`` [B, C_total] written in place.  Asynchronous."""
        batch, seq = token_ids.shape
        mask = self.full_mask() if task_mask is None else task_mask
        _check(lib().mt_forward(self.handle, _ptr(token_ids), _ptr(segment_ids), _ptr(lengths), mask, batch, seq,
                                _ptr(logits), _stream(stream)), "mt_forward", self.handle)

    def forward_tokens(self, token_ids, segment_ids, lengths, logits, token_logits, task_mask: Optional[int] = None,
                       stream=None) -> None:
        """forward() for trees with token-level tasks: ``logits`` [B, total_classes] (or None) and
        ``token_logits`` [B, S, total_token_classes] (or None), both fp32, written in place."""
        batch, seq = token_ids.shape
        mask = self.full_mask() if task_mask is None else task_mask
        _check(lib().mt_forward_tokens(self.handle, _ptr(token_ids), _ptr(segment_ids), _ptr(lengths), mask, batch, seq,
                                       _ptr(logits), _ptr(token_logits), None, _stream(stream)),
               "mt_forward_tokens", self.handle)

    def forward_events(self, token_ids, segment_ids, lengths, logits, task_events, task_mask: Optional[int] = None,
                       stream=None) -> None:
        """forward() that records ``task_events[t]`` (torch.cuda.Event or None per task) as soon as the
        launch writing task t's logits has been enqueued."""
        batch, seq = token_ids.shape
        mask = self.full_mask() if task_mask is None else task_mask
        handles = (_P * self.cfg.n_tasks)()
        for t, ev in enumerate(task_events):
            if ev is not None:
                if not ev.cuda_event:       # torch creates the event lazily
                    ev.record(torch_stream_for_init())
                handles[t] = ev.cuda_event
        _check(lib().mt_forward_events(self.handle, _ptr(token_ids), _ptr(segment_ids), _ptr(lengths), mask, batch,
                                       seq, _ptr(logits), handles, _stream(stream)), "mt_forward_events", self.handle)

    def forward_host(self, token_ids, segment_ids, lengths, logits, task_mask: Optional[int] = None,
                     stream=None) -> None:
        """Host (ideally pinned) int32 tensors in, host fp32 ``logits`` out; returns after the copy back."""
        batch, seq = token_ids.shape
        mask = self.full_mask() if task_mask is None else task_mask
        _check(lib().mt_forward_host(self.handle, _ptr(token_ids), _ptr(segment_ids), _ptr(lengths), mask, batch, seq,
                                     _ptr(logits), _stream(stream)), "mt_forward_host", self.handle)

    def forward_host_async(self, token_ids, segment_ids, lengths, logits, task_mask: Optional[int] = None,
                           stream=None) -> None:
        """forward_host without the final synchronisation (pinned host tensors; capturable in a CUDA graph)."""
        batch, seq = token_ids.shape
        mask = self.full_mask() if task_mask is None else task_mask
        _check(lib().mt_forward_host_async(self.handle, _ptr(token_ids), _ptr(segment_ids), _ptr(lengths), mask, batch,
                                           seq, _ptr(logits), _stream(stream)), "mt_forward_host_async", self.handle)

    def poll_status(self, stream=None) -> int:
        flags = C.c_uint32(0)
        rc = lib().mt_poll_status(self.handle, _stream(stream), C.byref(flags))
        if rc not in (MT_OK, -8):
            _check(rc, "mt_poll_status", self.handle)
        return flags.value

    def profile_read(self):
        """{class name: (milliseconds, launches)} since the last read (option "profile")."""
        ms = (C.c_double * len(KERNEL_CLASSES))()
        n = (C.c_int64 * len(KERNEL_CLASSES))()
        _check(lib().mt_profile_read(self.handle, ms, n), "mt_profile_read", self.handle)
        return {name: (ms[i], n[i]) for i, name in enumerate(KERNEL_CLASSES)}

    def debug_hidden(self, task: int, layer: int, batch: int, seq: int):
        import torch
        out = torch.empty(batch * seq, self.cfg.hidden, dtype=torch.bfloat16, device=self.device)
        _check(lib().mt_debug_copy_hidden(self.handle, task, layer, out.data_ptr(), _stream()), "mt_debug_copy_hidden",
               self.handle)
        return out

    def close(self) -> None:
        if self.handle:
            lib().mt_destroy(self.handle)
            self.handle = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
