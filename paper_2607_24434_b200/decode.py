"""Host loop of one exact DraftExpert decode step (Algorithm 1) over an offloaded layer stack.

Only orchestration lives here: every arithmetic step is a call into the library (``binding``): the drafter's
layers (Eq. 5, ``moe_draft_step_cached``), the draft LM head with its confidence (``spec_draft_token``), the
confidence-expansion stop rule (Sec. 3.4, ``dx_controller_propose``), prefetching of the newly predicted verifier
experts (Sec. 3.5, ``expert_cache_prefetch``), the verifier's layers (Eq. 4 over the block's expert union,
``moe_verify_block_cached``: wait for useful transfers, load misses on demand) and greedy exact acceptance
(``spec_accept``).  Attention is stubbed out as in the synthetic stack workloads (pre-norm residual MoE sub-layers
only), so a token's hidden states depend on its own embedding alone; the token chain runs through a seeded
embedding table.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from . import binding


class OffloadedDecoder:
    """Layers whose routed experts sit in a pinned host pool behind ``cache``; shared and draft experts resident.

    ``budget`` is B_i of Eq. 14: an int (fixed layer-expert budget) or ``"cache"`` (what is left of the cache's
    n_layers * slots pairs once the predictions accepted so far are counted: a candidate whose new pairs no longer fit
    is the one that is expensive to verify).  ``tau`` is the confidence threshold of Eq. 14."""

    def __init__(self, ctx: binding.Context, layers: Sequence[binding.Layer], cache: binding.ExpertCache,
                 emb: torch.Tensor, W_lm: torch.Tensor, k_max: int = 8, tau: float = 1.0, budget="cache",
                 native: bool = False):
        """``native``: steps that are not recorded run as one library call (``dx_decoder_step``: the same calls in
        the same order from a host loop inside the library, no interpreter between them)."""
        self.ctx, self.layers, self.cache = ctx, list(layers), cache
        self._native = binding.Decoder(ctx, layers, cache, emb, W_lm, k_max, tau,
                                       -1 if budget == "cache" else int(budget)) if native else None
        self.emb, self.W_lm = emb, W_lm
        self.k_max, self.tau, self.budget = k_max, tau, budget
        sh = self.layers[0].shape
        self.shape = sh
        self.controller = binding.Controller(len(self.layers), sh.n_experts)
        dev = emb.device
        H = sh.hidden
        # two alternating hidden buffers per phase (h_in and h_out of a residual layer must be distinct)
        self._hd = [torch.empty((1, H), device=dev), torch.empty((1, H), device=dev)]
        self._hv = [torch.empty((k_max, H), device=dev), torch.empty((k_max, H), device=dev)]
        self._dout = {"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device=dev),
                      "topk_w": torch.empty((sh.top_k,), dtype=torch.float32, device=dev)}

    def close(self) -> None:
        self.controller.close()
        if self._native is not None:
            self._native.close()

    def _budget_now(self) -> int:
        if self.budget == "cache":
            return len(self.layers) * self.cache.slots - self.controller.size()
        return int(self.budget)

    def step(self, t0: int, record: bool = False, scripted_accept: Optional[int] = None) -> Dict[str, object]:
        """One decode step from the last emitted token ``t0``.  Returns the drafted tokens, the accepted length,
        the tokens emitted and the next step's start token; with ``record`` also what a checker needs to replay
        the step (every layer's input rows, the routing the library used, the cache calls in order).
        ``scripted_accept``: take this accepted length (capped at the block length) instead of the comparison's
        -- for synthetic weights, whose random draft experts agree with the target almost never."""
        if self._native is not None and not record:
            return self._native.step(t0, scripted_accept)
        L = len(self.layers)
        trace: Dict[str, object] = {"draft": [], "verify": [], "cache_calls": []} if record else {}
        self.cache.begin_step()
        self.controller.reset()
        if record:
            trace["cache_calls"].append(("begin_step",))
        drafted: List[int] = []
        prev = int(t0)
        for i in range(self.k_max):
            # ---- draft v_i: the drafter's stack on the embedding of the previous token (Algorithm 1, "Draft v_i")
            h = self._hd[0]
            h.copy_(self.emb[prev].float().unsqueeze(0))
            pred, rows = [], []
            for l, layer in enumerate(self.layers):
                h_out = self._hd[(l + 1) & 1]
                if record:
                    rows.append(h.clone())
                out = binding.moe_draft_step_cached(layer, h, h_out, self._dout, residual=True)
                pred.append(out["host_ids"])
                if record:
                    trace["cache_calls"].append(("stage", l, [out["host_ids"][0]]))
                h = h_out
            tok, conf = binding.spec_draft_token(self.ctx, h, self.W_lm, rms_norm=True)
            v, q = int(tok.item()), float(conf.item())
            # ---- "Compute confidence q_i, predicted experts, marginal expansion; stop drafting if ..."
            budget = self._budget_now()
            stop, delta, new = self.controller.propose(pred, q, self.tau, budget)
            if record:
                trace["draft"].append({"prev": prev, "rows": rows, "final": h.clone(), "pred": pred, "token": v, "q": q,
                                       "budget": budget, "stop": stop, "delta": delta, "new": new})
            if stop:
                break
            drafted.append(v)
            # ---- "Launch non-blocking prefetch for U_hat_i \\ (C u P)"
            by_layer: Dict[int, List[int]] = {}
            for (l, e) in new:
                by_layer.setdefault(l, []).append(e)
            for l in sorted(by_layer):
                self.cache.prefetch(l, by_layer[l])
                if record:
                    trace["cache_calls"].append(("prefetch", l, by_layer[l]))
            prev = v
        # ---- verify D with the full target MoE: rows are the inputs that predict d_1 .. d_K
        K = max(1, len(drafted))
        inputs = [int(t0)] + drafted[:K - 1]
        hv = self._hv[0][:K]
        hv.copy_(self.emb[torch.tensor(inputs, device=self.emb.device)].float())
        union_sizes: List[int] = []
        for l, layer in enumerate(self.layers):
            hv_out = self._hv[(l + 1) & 1][:K]
            if record:
                rows_in = hv.clone()
            out = binding.moe_verify_block_cached(layer, self.cache, l, hv, hv_out, residual=True)
            union_sizes.append(len(out["union_list"]))
            if record:
                trace["verify"].append({"rows": rows_in, "out": hv_out.clone(), "topk_ids": out["topk_ids"].clone(),
                                        "topk_w": out["topk_w"].clone(), "union": out["union_list"]})
                trace["cache_calls"].append(("stage_union", l, out["union_list"]))
            hv = hv_out
        draft_dev = torch.tensor(drafted if drafted else [-1], dtype=torch.int32, device=hv.device)
        acc = binding.spec_accept(self.ctx, hv, self.W_lm, draft_dev, rms_norm=True)
        target = acc["target"].tolist()
        n = int(acc["n_accept"].item()) if drafted else 0
        if scripted_accept is not None:
            n = min(int(scripted_accept), len(drafted))
        # "Accept the target-consistent prefix": d_1 .. d_n, then the target's own token for position n + 1 if a
        # row is left for it (with the whole block accepted the next step starts from d_K)
        emitted = drafted[:n] + ([target[n]] if n < K else [])
        res = {"drafted": drafted, "n_accept": n, "emitted": emitted, "next": emitted[-1], "target": target,
               "block_rows": K, "final": hv, "union_sizes": union_sizes}
        if record:
            res["trace"] = trace
        return res
