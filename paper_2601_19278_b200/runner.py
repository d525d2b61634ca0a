"""Convenience driver around the binding: places one workload's synthetic inputs on the GPU,
allocates the output buffers and runs dart_draft_step + dart_build_tree.  Used by the tests,
the smoke check and the benchmark; it performs no arithmetic of its own."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding, synthetic


class DraftSession:
    def __init__(self, w: synthetic.Workload, weights: Dict[str, torch.Tensor], ngram: Optional[Dict[str, np.ndarray]],
                 device: str = "cuda:0", want_logits: bool = False, **cfg_over):
        self.w = w
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.cfg = binding.make_config(w, **cfg_over)
        self.weights = {k: v.to(self.dev) for k, v in weights.items()}
        self.draft = binding.DartDraft(self.cfg, self.weights, ngram)
        B, K, k, bud = w.batch, w.K, self.cfg.topk, self.cfg.tree_budget
        i32 = dict(dtype=torch.int32, device=self.dev)
        self.topk_ids = torch.full((B, K, k), -7, **i32)
        self.topk_slogit = torch.zeros((B, K, k), dtype=torch.float32, device=self.dev)
        self.logits = torch.zeros((B, K, w.vocab), dtype=torch.float32, device=self.dev) if want_logits else None
        self.tokens = torch.full((B, bud), -7, **i32)
        self.parents = torch.full((B, bud), -7, **i32)
        self.depth = torch.full((B, bud), -7, **i32)
        self.mask = torch.full((B, bud, bud), 9, dtype=torch.uint8, device=self.dev)
        self.n_nodes = torch.zeros((B,), **i32)
        self.scores = torch.zeros((B, bud), dtype=torch.float32, device=self.dev)
        self.inp = None

    def load_inputs(self, inp: Dict[str, object]) -> None:
        """Copy one step's inputs (synthetic.make_step_inputs) to the device."""
        d = self.dev
        self.inp = {
            "feats": inp["feats"].to(d), "tokens": inp["tokens"].to(d), "seq_lens": inp["seq_lens"].to(d),
            "seq_lens_host": inp["seq_lens"].numpy().astype(np.int32), "k_cache": inp["k_cache"].to(d),
            "v_cache": inp["v_cache"].to(d), "ctx_tail": inp["ctx_tail"].to(d), "n_fresh": int(inp["n_fresh"]),
        }

    def step(self, step_counter: int = 0, stream=None) -> None:
        i = self.inp
        self.draft.draft_step(feats=i["feats"] if i["n_fresh"] else None, tokens=i["tokens"] if i["n_fresh"] else None,
                              seq_lens=i["seq_lens"], seq_lens_host=i["seq_lens_host"], k_cache=i["k_cache"],
                              v_cache=i["v_cache"], n_fresh=i["n_fresh"], topk_ids=self.topk_ids,
                              topk_slogit=self.topk_slogit, logits=self.logits, step_counter=step_counter, stream=stream)

    def tree(self, stream=None, topk_ids=None, topk_slogit=None, ctx_tail=None, first_row: Optional[int] = None) -> None:
        fr = max(self.inp["n_fresh"], 1) - 1 if first_row is None else first_row
        self.draft.build_tree(batch=self.w.batch, topk_ids=self.topk_ids if topk_ids is None else topk_ids,
                              topk_slogit=self.topk_slogit if topk_slogit is None else topk_slogit,
                              ctx_tail=self.inp["ctx_tail"] if ctx_tail is None else ctx_tail,
                              tokens=self.tokens, parents=self.parents, depth=self.depth, mask=self.mask,
                              n_nodes=self.n_nodes, scores=self.scores, first_row=fr, stream=stream)

    def tree_outputs(self) -> Dict[str, np.ndarray]:
        torch.cuda.synchronize(self.dev)
        return {"tokens": self.tokens.cpu().numpy(), "parents": self.parents.cpu().numpy(),
                "depth": self.depth.cpu().numpy(), "mask": self.mask.cpu().numpy(),
                "n_nodes": self.n_nodes.cpu().numpy(), "scores": self.scores.cpu().numpy()}

    def close(self):
        self.draft.close()
