"""Thin ctypes binding of ``libdart.so`` (the C ABI declared in ``include/dart.h``).

Argument marshalling only: torch provides device memory and streams, every step of the
drafting path runs in the library's CUDA kernels.  There is no fallback: if the shared
library is missing or fails to load, importing callers get an exception.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DART_LIB: load another build of the same library instead (the tests run once against the -DDART_DEBUG build)
LIB_PATH = os.environ.get("DART_LIB") or os.path.join(_HERE, "libdart.so")

DART_OK = 0
DART_ERR_INVALID_ARG = -1
DART_ERR_UNSUPPORTED_ARCH = -2
DART_ERR_CUDA = -3
DART_ERR_CAPACITY = -4
DART_ERR_TIMEOUT = -5
DART_ERR_INTERNAL = -6

EXPORTS = [
    "dart_draft_init", "dart_draft_step", "dart_build_tree", "dart_draft_destroy", "dart_last_device_status",
    "dart_last_cuda_error", "dart_status_string", "dart_workspace_bytes", "dart_ngram_bytes", "dart_train_attention_fwd", "dart_step_launch_count", "dart_draft_prefill", "dart_tree_verify_inputs",
    "dart_set_profile_events", "dart_topk_rows_noalloc", "dart_selftest_bounded_wait", "dart_draft_step_host",
]


class DartConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("mlp_inter", C.c_int32), ("vocab", C.c_int32), ("feat_in", C.c_int32),
        ("max_batch", C.c_int32), ("max_prefix", C.c_int32), ("K", C.c_int32), ("topk", C.c_int32),
        ("beam", C.c_int32), ("tree_budget", C.c_int32), ("ngram_order", C.c_int32),
        ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("w_ng", C.c_float), ("logit_decay", C.c_float),
        ("level_exp", C.c_float), ("eps_logit", C.c_float), ("eps_ng", C.c_float), ("temperature", C.c_float),
        ("philox_seed", C.c_uint64), ("ngram_layout", C.c_int32), ("reserved0", C.c_int32),
    ]


NGRAM_HASH, NGRAM_TRIE = 0, 1


class DartTrainAttnIn(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("prompt_len", C.c_int32), ("draft_len", C.c_int32), ("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p),
                ("seq_lens_host", C.c_void_p), ("out", C.c_void_p), ("status", C.c_void_p)]


WEIGHT_NAMES = ["w_fc", "embed", "mask_vec", "norm_g", "norm_e", "w_q", "w_k", "w_v", "w_o", "norm_post",
                "w_gate", "w_up", "w_down", "norm_final", "w_lm"]


class DartWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


class DartNgramHost(C.Structure):
    _fields_ = [("n_rows", C.c_int64), ("order", C.c_void_p), ("ctx0", C.c_void_p), ("ctx1", C.c_void_p),
                ("next", C.c_void_p), ("score", C.c_void_p)]


class DartStepIn(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_fresh", C.c_int32), ("feats", C.c_void_p), ("tokens", C.c_void_p),
                ("seq_lens", C.c_void_p), ("seq_lens_host", C.c_void_p), ("k_cache", C.c_void_p),
                ("v_cache", C.c_void_p), ("step_counter", C.c_uint64), ("fresh_counts_host", C.c_void_p)]


class DartPrefillIn(C.Structure):
    _fields_ = [("batch", C.c_int32), ("feats", C.c_void_p), ("tokens", C.c_void_p), ("seq_lens_host", C.c_void_p),
                ("new_rows_host", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p)]


class DartVerifyIn(C.Structure):
    _fields_ = [("batch", C.c_int32), ("max_levels", C.c_int32), ("parents", C.c_void_p), ("depth", C.c_void_p),
                ("n_nodes", C.c_void_p), ("root_pos", C.c_void_p)]


class DartVerifyOut(C.Structure):
    _fields_ = [("position_ids", C.c_void_p), ("retrieve", C.c_void_p), ("n_leaves", C.c_void_p)]


class DartStepOut(C.Structure):
    _fields_ = [("topk_ids", C.c_void_p), ("topk_slogit", C.c_void_p), ("logits", C.c_void_p)]


class DartTreeIn(C.Structure):
    _fields_ = [("batch", C.c_int32), ("first_row", C.c_int32), ("n_levels", C.c_int32), ("topk_ids", C.c_void_p),
                ("topk_slogit", C.c_void_p), ("ctx_tail", C.c_void_p), ("first_rows_host", C.c_void_p)]


class DartTreeOut(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("parents", C.c_void_p), ("depth", C.c_void_p), ("mask", C.c_void_p),
                ("n_nodes", C.c_void_p), ("scores", C.c_void_p)]


class DartHostIo(C.Structure):
    _fields_ = [("in_host", C.c_void_p), ("in_dev", C.c_void_p), ("in_bytes", C.c_size_t),
                ("out_dev", C.c_void_p), ("out_host", C.c_void_p), ("out_bytes", C.c_size_t)]


_lib = None


def lib() -> C.CDLL:
    """Load libdart.so (once).  Raises if it has not been built: there is no CPU fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_19278_b200.build` "
                               "(the drafting step has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.dart_draft_init.argtypes = [C.POINTER(DartConfig), C.POINTER(DartWeights), C.POINTER(DartNgramHost),
                                      C.POINTER(C.c_void_p)]
        L.dart_draft_init.restype = C.c_int
        L.dart_draft_step.argtypes = [C.c_void_p, C.POINTER(DartStepIn), C.POINTER(DartStepOut), C.c_void_p]
        L.dart_draft_step.restype = C.c_int
        L.dart_build_tree.argtypes = [C.c_void_p, C.POINTER(DartTreeIn), C.POINTER(DartTreeOut), C.c_void_p]
        L.dart_build_tree.restype = C.c_int
        L.dart_draft_step_host.argtypes = [C.c_void_p, C.POINTER(DartHostIo), C.POINTER(DartStepIn), C.POINTER(DartStepOut),
                                           C.POINTER(DartTreeIn), C.POINTER(DartTreeOut), C.c_void_p]
        L.dart_draft_step_host.restype = C.c_int
        L.dart_draft_destroy.argtypes = [C.c_void_p]
        L.dart_draft_destroy.restype = C.c_int
        L.dart_last_device_status.argtypes = [C.c_void_p, C.c_void_p]
        L.dart_last_device_status.restype = C.c_int
        L.dart_last_cuda_error.argtypes = [C.c_void_p]
        L.dart_last_cuda_error.restype = C.c_int
        L.dart_status_string.argtypes = [C.c_int]
        L.dart_status_string.restype = C.c_char_p
        L.dart_workspace_bytes.argtypes = [C.POINTER(DartConfig)]
        L.dart_workspace_bytes.restype = C.c_size_t
        L.dart_train_attention_fwd.argtypes = [C.POINTER(DartTrainAttnIn), C.c_void_p]
        L.dart_train_attention_fwd.restype = C.c_int
        L.dart_ngram_bytes.argtypes = [C.c_void_p]
        L.dart_ngram_bytes.restype = C.c_size_t
        L.dart_tree_verify_inputs.argtypes = [C.c_void_p, C.POINTER(DartVerifyIn), C.POINTER(DartVerifyOut), C.c_void_p]
        L.dart_tree_verify_inputs.restype = C.c_int
        L.dart_draft_prefill.argtypes = [C.c_void_p, C.POINTER(DartPrefillIn), C.c_void_p]
        L.dart_draft_prefill.restype = C.c_int
        L.dart_step_launch_count.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.dart_step_launch_count.restype = C.c_int
        L.dart_set_profile_events.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.dart_set_profile_events.restype = C.c_int
        L.dart_topk_rows_noalloc.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p,
                                             C.c_void_p, C.c_void_p]
        L.dart_topk_rows_noalloc.restype = C.c_int
        L.dart_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        L.dart_selftest_bounded_wait.restype = C.c_int
        _lib = L
    return _lib


class DartError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        name = lib().dart_status_string(status).decode()
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{where}: {name}{extra}")


def make_config(w, **over) -> DartConfig:
    """dart_config from a synthetic.Workload (Appendix D defaults for the pruning constants)."""
    cfg = DartConfig()
    cfg.struct_size = C.sizeof(DartConfig)
    vals = dict(hidden=w.hidden, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                mlp_inter=w.mlp_inter, vocab=w.vocab, feat_in=w.feat_in, max_batch=w.batch,
                max_prefix=w.max_prefix, K=w.K, topk=w.topk, beam=w.beam, tree_budget=w.tree_budget,
                ngram_order=3, rope_theta=1e6, rms_eps=1e-6, w_ng=0.5, logit_decay=0.9, level_exp=0.7,
                eps_logit=1e-10, eps_ng=1e-10, temperature=w.temperature, philox_seed=1234,
                ngram_layout=NGRAM_HASH)
    vals.update(over)
    for k, v in vals.items():
        setattr(cfg, k, v)
    return cfg


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


class DartDraft:
    """Owner of a dart_handle.  Methods mirror the C entry points one to one."""

    def __init__(self, cfg: DartConfig, weights: Dict[str, torch.Tensor], ngram: Optional[Dict[str, np.ndarray]] = None):
        self._h = C.c_void_p()
        self.cfg = cfg
        names = [n for n in WEIGHT_NAMES if not (n == "w_fc" and cfg.feat_in == 0)]   # no fusion matrix without a feature FC
        self._weights = {n: weights[n] for n in names}             # keep the device tensors alive
        for n, t in self._weights.items():
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous(), n
        ws = DartWeights(**{n: t.data_ptr() for n, t in self._weights.items()})
        ng = None
        if ngram is not None and len(ngram["next"]):
            self._ng = {k: np.ascontiguousarray(v) for k, v in ngram.items()}
            assert self._ng["order"].dtype == np.uint8 and self._ng["score"].dtype == np.float32
            ng = DartNgramHost(len(self._ng["next"]), self._ng["order"].ctypes.data, self._ng["ctx0"].ctypes.data,
                               self._ng["ctx1"].ctypes.data, self._ng["next"].ctypes.data, self._ng["score"].ctypes.data)
        rc = lib().dart_draft_init(C.byref(cfg), C.byref(ws), C.byref(ng) if ng is not None else None, C.byref(self._h))
        if rc != DART_OK:
            raise DartError(rc, "dart_draft_init", lib().dart_last_cuda_error(None))

    def close(self):
        if self._h:
            lib().dart_draft_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _stream(stream) -> int:
        return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream

    def draft_step(self, *, feats, tokens, seq_lens, seq_lens_host: np.ndarray, k_cache, v_cache, n_fresh,
                   topk_ids, topk_slogit, logits=None, step_counter: int = 0, stream=None) -> None:
        """dart_draft_step: all tensors are caller-owned device tensors; seq_lens_host is a host int32 array.
        n_fresh: one count for all sequences, or a sequence of per-sequence counts (fresh_counts_host)."""
        slh = np.ascontiguousarray(seq_lens_host, dtype=np.int32)
        counts = None if isinstance(n_fresh, (int, np.integer)) else np.ascontiguousarray(n_fresh, dtype=np.int32)
        sin = DartStepIn(len(slh), int(n_fresh) if counts is None else int(counts.max(initial=0)), _ptr(feats), _ptr(tokens),
                         _ptr(seq_lens), slh.ctypes.data, _ptr(k_cache), _ptr(v_cache), step_counter,
                         None if counts is None else counts.ctypes.data)
        sout = DartStepOut(_ptr(topk_ids), _ptr(topk_slogit), _ptr(logits))
        rc = lib().dart_draft_step(self._h, C.byref(sin), C.byref(sout), self._stream(stream))
        if rc != DART_OK:
            raise DartError(rc, "dart_draft_step", lib().dart_last_cuda_error(self._h))

    def host_step(self, *, in_host, in_dev, out_host, out_dev, feats, tokens, seq_lens, seq_lens_host, k_cache, v_cache,
                  n_fresh, topk_ids, topk_slogit, ctx_tail, tree_tokens, parents, depth, mask, n_nodes, scores=None,
                  logits=None, first_row=0, n_levels: Optional[int] = None, stream=None) -> "HostStep":
        """dart_draft_step_host with its argument structures built once: the returned object is called with the
        step counter and runs copy in, forward pass, tree, copy out, wait.  in_host / out_host are (pinned) host byte
        tensors, in_dev / out_dev the device buffers that the device tensors passed here are views of."""
        return HostStep(self, dict(in_host=in_host, in_dev=in_dev, out_host=out_host, out_dev=out_dev, feats=feats,
                                   tokens=tokens, seq_lens=seq_lens, seq_lens_host=seq_lens_host, k_cache=k_cache,
                                   v_cache=v_cache, n_fresh=n_fresh, topk_ids=topk_ids, topk_slogit=topk_slogit,
                                   ctx_tail=ctx_tail, tree_tokens=tree_tokens, parents=parents, depth=depth, mask=mask,
                                   n_nodes=n_nodes, scores=scores, logits=logits, first_row=first_row,
                                   n_levels=n_levels), stream)

    def prefill(self, *, feats, tokens, seq_lens_host, new_rows_host, k_cache, v_cache, stream=None) -> None:
        """dart_draft_prefill: append the k, v of new prefix rows (packed features / next-token ids) to the caches."""
        slh = np.ascontiguousarray(seq_lens_host, dtype=np.int32)
        nrh = np.ascontiguousarray(new_rows_host, dtype=np.int32)
        pin = DartPrefillIn(len(slh), _ptr(feats), _ptr(tokens), slh.ctypes.data, nrh.ctypes.data, _ptr(k_cache), _ptr(v_cache))
        rc = lib().dart_draft_prefill(self._h, C.byref(pin), self._stream(stream))
        if rc != DART_OK:
            raise DartError(rc, "dart_draft_prefill", lib().dart_last_cuda_error(self._h))

    def verify_inputs(self, *, batch: int, max_levels: int, parents, depth, n_nodes, root_pos, position_ids, retrieve, n_leaves,
                      stream=None) -> None:
        """dart_tree_verify_inputs: position ids and root-to-leaf paths of the trees dart_build_tree wrote."""
        vin = DartVerifyIn(batch, max_levels, _ptr(parents), _ptr(depth), _ptr(n_nodes), _ptr(root_pos))
        vout = DartVerifyOut(_ptr(position_ids), _ptr(retrieve), _ptr(n_leaves))
        rc = lib().dart_tree_verify_inputs(self._h, C.byref(vin), C.byref(vout), self._stream(stream))
        if rc != DART_OK:
            raise DartError(rc, "dart_tree_verify_inputs", lib().dart_last_cuda_error(self._h))

    def build_tree(self, *, batch: int, topk_ids, topk_slogit, ctx_tail, tokens, parents, depth, mask, n_nodes,
                   scores=None, first_row=0, n_levels: Optional[int] = None, stream=None) -> None:
        """dart_build_tree on caller-owned device tensors.  first_row: one row for all sequences, or a sequence
        of per-sequence first rows (first_rows_host)."""
        rows = None if isinstance(first_row, (int, np.integer)) else np.ascontiguousarray(first_row, dtype=np.int32)
        fr = int(first_row) if rows is None else int(rows.min())
        tin = DartTreeIn(batch, fr, self.cfg.K - fr if n_levels is None else n_levels,
                         _ptr(topk_ids), _ptr(topk_slogit), _ptr(ctx_tail), None if rows is None else rows.ctypes.data)
        tout = DartTreeOut(_ptr(tokens), _ptr(parents), _ptr(depth), _ptr(mask), _ptr(n_nodes), _ptr(scores))
        rc = lib().dart_build_tree(self._h, C.byref(tin), C.byref(tout), self._stream(stream))
        if rc != DART_OK:
            raise DartError(rc, "dart_build_tree", lib().dart_last_cuda_error(self._h))

    def device_status(self, stream=None) -> int:
        return lib().dart_last_device_status(self._h, self._stream(stream))

    def selftest_bounded_wait(self, spin_limit: int, leave_ticket: bool = False, stream=None) -> None:
        """dart_selftest_bounded_wait: enqueue a wait that runs out on purpose (device_status() then reports the time-out)."""
        rc = lib().dart_selftest_bounded_wait(self._h, spin_limit, 1 if leave_ticket else 0, self._stream(stream))
        if rc != DART_OK:
            raise DartError(rc, "dart_selftest_bounded_wait", lib().dart_last_cuda_error(self._h))

    def set_profile_events(self, stage: int, start: torch.cuda.Event, stop: torch.cuda.Event) -> None:
        """dart_set_profile_events: bracket one stage of the next call with two torch CUDA events."""
        rc = lib().dart_set_profile_events(self._h, stage, start.cuda_event, stop.cuda_event)
        if rc != DART_OK:
            raise DartError(rc, "dart_set_profile_events")

    def launch_count(self, batch: int, n_fresh: int) -> int:
        return lib().dart_step_launch_count(self._h, batch, n_fresh)

    def ngram_bytes(self) -> int:
        return lib().dart_ngram_bytes(self._h)


def topk_rows_noalloc(logits: torch.Tensor, topk: int, eps_logit: float, out_ids: torch.Tensor, out_slogit: torch.Tensor,
                      stream=None) -> None:
    """dart_topk_rows_noalloc: log-softmax + top-k of fp32 logits [rows, vocab] into caller-owned outputs.
    For callers that may not allocate device memory: the library uses a fixed scratch array of its own
    (at most 128 rows; calls on one GPU must not overlap)."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous() and logits.dim() == 2
    rows, vocab = logits.shape
    st = (stream if stream is not None else torch.cuda.current_stream()).cuda_stream
    rc = lib().dart_topk_rows_noalloc(logits.data_ptr(), rows, vocab, topk, eps_logit, out_ids.data_ptr(),
                                      out_slogit.data_ptr(), st)
    if rc != DART_OK:
        raise DartError(rc, "dart_topk_rows_noalloc")


def train_attention_fwd(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_lens, prompt_len: int, draft_len: int,
                        out: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None) -> None:
    """dart_train_attention_fwd on caller-owned device tensors: q [B, Hq, L, dh], k, v [B, Hkv, L, dh] bf16,
    L = prompt_len * (1 + draft_len); seq_lens: host ints [B]."""
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    a = DartTrainAttnIn(batch=q.shape[0], n_q_heads=q.shape[1], n_kv_heads=k.shape[1], head_dim=q.shape[3], prompt_len=prompt_len,
                        draft_len=draft_len, q=q.data_ptr(), k=k.data_ptr(), v=v.data_ptr(), seq_lens_host=lens.ctypes.data,
                        out=out.data_ptr(), status=_ptr(status))
    st = stream if stream is not None else torch.cuda.current_stream(q.device)
    rc = lib().dart_train_attention_fwd(C.byref(a), C.c_void_p(st.cuda_stream))
    if rc != DART_OK:
        raise DartError(rc, "dart_train_attention_fwd", lib().dart_last_cuda_error(None))


def workspace_bytes(cfg: DartConfig) -> int:
    return lib().dart_workspace_bytes(C.byref(cfg))


class HostStep:
    """One prepared dart_draft_step_host call (argument marshalling only; see DartDraft.host_step)."""

    def __init__(self, draft: "DartDraft", a: dict, stream) -> None:
        self._draft, self._keep = draft, a
        self._slh = np.ascontiguousarray(a["seq_lens_host"], dtype=np.int32)
        nf = a["n_fresh"]
        self._counts = None if isinstance(nf, (int, np.integer)) else np.ascontiguousarray(nf, dtype=np.int32)
        fr = a["first_row"]
        self._rows = None if isinstance(fr, (int, np.integer)) else np.ascontiguousarray(fr, dtype=np.int32)
        B = len(self._slh)
        any_fresh = (int(nf) if self._counts is None else int(self._counts.max(initial=0))) > 0
        self.io = DartHostIo(_ptr(a["in_host"]), _ptr(a["in_dev"]), a["in_host"].numel() * a["in_host"].element_size(),
                             _ptr(a["out_dev"]), _ptr(a["out_host"]), a["out_host"].numel() * a["out_host"].element_size())
        self.sin = DartStepIn(B, int(nf) if self._counts is None else int(self._counts.max(initial=0)),
                              _ptr(a["feats"]) if any_fresh else None, _ptr(a["tokens"]) if any_fresh else None,
                              _ptr(a["seq_lens"]), self._slh.ctypes.data, _ptr(a["k_cache"]), _ptr(a["v_cache"]), 0,
                              None if self._counts is None else self._counts.ctypes.data)
        self.sout = DartStepOut(_ptr(a["topk_ids"]), _ptr(a["topk_slogit"]), _ptr(a["logits"]))
        f0 = int(fr) if self._rows is None else int(self._rows.min())
        self.tin = DartTreeIn(B, f0, draft.cfg.K - f0 if a["n_levels"] is None else a["n_levels"], _ptr(a["topk_ids"]),
                              _ptr(a["topk_slogit"]), _ptr(a["ctx_tail"]), None if self._rows is None else self._rows.ctypes.data)
        self.tout = DartTreeOut(_ptr(a["tree_tokens"]), _ptr(a["parents"]), _ptr(a["depth"]), _ptr(a["mask"]),
                                _ptr(a["n_nodes"]), _ptr(a["scores"]))
        self._st = draft._stream(stream)
        self._fn = lib().dart_draft_step_host
        self._args = (draft._h, C.byref(self.io), C.byref(self.sin), C.byref(self.sout), C.byref(self.tin), C.byref(self.tout),
                      self._st)

    def __call__(self, step_counter: int = 0) -> None:
        self.sin.step_counter = step_counter
        rc = self._fn(*self._args)
        if rc != DART_OK:
            raise DartError(rc, "dart_draft_step_host", lib().dart_last_cuda_error(self._draft._h))
