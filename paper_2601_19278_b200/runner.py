"""Convenience driver around the binding: places one workload's synthetic inputs on the GPU,
allocates the output buffers and runs dart_draft_step + dart_build_tree.  Used by the tests,
the smoke check and the benchmark; it performs no arithmetic of its own."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding, synthetic


GUARD = 64   # sentinel elements in front of and behind every output buffer


class DraftSession:
    """Every output buffer sits between two runs of sentinel elements; check_guards() (called by tree_outputs() and
    close()) fails if a kernel wrote outside the buffer it was given."""

    def __init__(self, w: synthetic.Workload, weights: Dict[str, torch.Tensor], ngram: Optional[Dict[str, np.ndarray]],
                 device: str = "cuda:0", want_logits: bool = False, **cfg_over):
        self.w = w
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.cfg = binding.make_config(w, **cfg_over)
        self.weights = {k: v.to(self.dev) for k, v in weights.items()}
        self.draft = binding.DartDraft(self.cfg, self.weights, ngram)
        B, K, k, bud = w.batch, w.K, self.cfg.topk, self.cfg.tree_budget
        self._guards = []
        self.topk_ids = self._guarded((B, K, k), torch.int32, -7)
        self.topk_slogit = self._guarded((B, K, k), torch.float32, 0)
        self.logits = self._guarded((B, K, w.vocab), torch.float32, 0) if want_logits else None
        self.tokens = self._guarded((B, bud), torch.int32, -7)
        self.parents = self._guarded((B, bud), torch.int32, -7)
        self.depth = self._guarded((B, bud), torch.int32, -7)
        self.mask = self._guarded((B, bud, bud), torch.uint8, 9)
        self.n_nodes = self._guarded((B,), torch.int32, 0)
        self.scores = self._guarded((B, bud), torch.float32, 0)
        self.inp = None

    _SENTINEL = {torch.int32: 0x5A5A5A5A, torch.float32: 1.2345e30, torch.uint8: 0xA5}

    def _guarded(self, shape, dtype, fill) -> torch.Tensor:
        n = int(np.prod(shape))
        buf = torch.full((n + 2 * GUARD,), self._SENTINEL[dtype], dtype=dtype, device=self.dev)
        view = buf[GUARD:GUARD + n].view(shape)
        view.fill_(fill)
        self._guards.append((buf, n))
        return view

    def check_guards(self) -> None:
        """The sentinels around every output buffer are intact: no kernel wrote before or behind its output."""
        torch.cuda.synchronize(self.dev)
        for buf, n in self._guards:
            want = torch.tensor(self._SENTINEL[buf.dtype], dtype=buf.dtype, device=self.dev)
            assert bool((buf[:GUARD] == want).all()) and bool((buf[GUARD + n:] == want).all()), \
                f"a kernel wrote outside a {buf.dtype} output buffer of {n} elements"

    def load_inputs(self, inp: Dict[str, object]) -> None:
        """Copy one step's inputs (synthetic.make_step_inputs) to the device."""
        d = self.dev
        self.inp = {
            "feats": inp["feats"].to(d), "tokens": inp["tokens"].to(d), "seq_lens": inp["seq_lens"].to(d),
            "seq_lens_host": inp["seq_lens"].numpy().astype(np.int32), "k_cache": inp["k_cache"].to(d),
            "v_cache": inp["v_cache"].to(d), "ctx_tail": inp["ctx_tail"].to(d),
            # one count for all sequences, or a list of per-sequence counts
            "n_fresh": inp["n_fresh"] if isinstance(inp["n_fresh"], (list, tuple, np.ndarray)) else int(inp["n_fresh"]),
        }

    def pack_io(self):
        """Re-home the step's small inputs (features, tokens, lengths, context tail) in ONE device buffer and
        the tree outputs in another, each with a pinned host mirror, so that a caller moves a step's inputs
        and results with one copy each way.  Returns (in_host, in_dev, out_host, out_dev, host_views): the
        byte buffers and the host-side views of every field."""
        def layout(fields):
            off, spec = 0, {}
            for name, t in fields:
                off = (off + 255) // 256 * 256
                spec[name] = (off, t.numel() * t.element_size(), t.dtype, tuple(t.shape))
                off += t.numel() * t.element_size()
            return spec, (off + 255) // 256 * 256

        def carve(buf, spec):
            return {n: buf[o:o + nb].view(dt).view(shape) for n, (o, nb, dt, shape) in spec.items()}

        in_fields = [(n, self.inp[n]) for n in ("feats", "tokens", "seq_lens", "ctx_tail")]
        out_fields = [(n, getattr(self, n)) for n in ("tokens", "parents", "depth", "mask", "n_nodes")]
        ispec, ibytes = layout(in_fields)
        ospec, obytes = layout(out_fields)
        in_dev = torch.zeros(ibytes, dtype=torch.uint8, device=self.dev)
        out_dev = torch.zeros(obytes, dtype=torch.uint8, device=self.dev)
        in_host = torch.zeros(ibytes, dtype=torch.uint8).pin_memory()
        out_host = torch.zeros(obytes, dtype=torch.uint8).pin_memory()
        dviews, hviews = carve(in_dev, ispec), carve(in_host, ispec)
        for n, t in in_fields:
            hviews[n].copy_(t.cpu())
            dviews[n].copy_(t)
            self.inp[n] = dviews[n]
        oviews = carve(out_dev, ospec)
        for n, t in out_fields:
            oviews[n].copy_(t)
            setattr(self, n, oviews[n])
        hviews.update({"out_" + n: v for n, v in carve(out_host, ospec).items()})
        return in_host, in_dev, out_host, out_dev, hviews

    def step(self, step_counter: int = 0, stream=None) -> None:
        i = self.inp
        any_fresh = int(np.max(i["n_fresh"])) > 0
        self.draft.draft_step(feats=i["feats"] if any_fresh else None, tokens=i["tokens"] if any_fresh else None,
                              seq_lens=i["seq_lens"], seq_lens_host=i["seq_lens_host"], k_cache=i["k_cache"],
                              v_cache=i["v_cache"], n_fresh=i["n_fresh"], topk_ids=self.topk_ids,
                              topk_slogit=self.topk_slogit, logits=self.logits, step_counter=step_counter, stream=stream)

    def prefill(self, feats: torch.Tensor, tokens: torch.Tensor, new_rows, stream=None) -> None:
        """dart_draft_prefill on this session's caches: new_rows[b] rows are appended after the current lengths,
        which the caller then advances (self.inp["seq_lens"], self.inp["seq_lens_host"])."""
        self.draft.prefill(feats=feats.to(self.dev), tokens=tokens.to(self.dev), seq_lens_host=self.inp["seq_lens_host"],
                           new_rows_host=np.asarray(new_rows, dtype=np.int32), k_cache=self.inp["k_cache"],
                           v_cache=self.inp["v_cache"], stream=stream)

    def tree(self, stream=None, topk_ids=None, topk_slogit=None, ctx_tail=None, first_row: Optional[int] = None) -> None:
        nf = self.inp["n_fresh"]
        if first_row is not None:
            fr = first_row
        elif isinstance(nf, int):
            fr = max(nf, 1) - 1
        else:
            fr = [max(int(f), 1) - 1 for f in nf]      # level 0 of sequence b = its last fresh row
        self.draft.build_tree(batch=self.w.batch, topk_ids=self.topk_ids if topk_ids is None else topk_ids,
                              topk_slogit=self.topk_slogit if topk_slogit is None else topk_slogit,
                              ctx_tail=self.inp["ctx_tail"] if ctx_tail is None else ctx_tail,
                              tokens=self.tokens, parents=self.parents, depth=self.depth, mask=self.mask,
                              n_nodes=self.n_nodes, scores=self.scores, first_row=fr, stream=stream)

    def host_step(self, in_host, in_dev, out_host, out_dev, stream=None):
        """A prepared dart_draft_step_host call over the buffers pack_io returned: call it with the step counter."""
        i, nf = self.inp, self.inp["n_fresh"]
        fr = max(nf, 1) - 1 if isinstance(nf, int) else [max(int(f), 1) - 1 for f in nf]
        return self.draft.host_step(in_host=in_host, in_dev=in_dev, out_host=out_host, out_dev=out_dev, feats=i["feats"],
                                    tokens=i["tokens"], seq_lens=i["seq_lens"], seq_lens_host=i["seq_lens_host"],
                                    k_cache=i["k_cache"], v_cache=i["v_cache"], n_fresh=nf, topk_ids=self.topk_ids,
                                    topk_slogit=self.topk_slogit, ctx_tail=i["ctx_tail"], tree_tokens=self.tokens,
                                    parents=self.parents, depth=self.depth, mask=self.mask, n_nodes=self.n_nodes,
                                    scores=self.scores, logits=self.logits, first_row=fr, stream=stream)

    def tree_outputs(self) -> Dict[str, np.ndarray]:
        self.check_guards()
        return {"tokens": self.tokens.cpu().numpy(), "parents": self.parents.cpu().numpy(),
                "depth": self.depth.cpu().numpy(), "mask": self.mask.cpu().numpy(),
                "n_nodes": self.n_nodes.cpu().numpy(), "scores": self.scores.cpu().numpy()}

    def close(self):
        if self._guards:
            self.check_guards()
            self._guards = []
        self.draft.close()
