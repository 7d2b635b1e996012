"""A rollout state built the way a framework user would: named torch CPU tensors, ``chunk`` for the
tensor-parallel slices and ``cat`` for the fusions.  Used to pin the oracle to library routines; it
contains no flat-offset arithmetic beyond concatenating the tensors in their canonical order."""
from collections import OrderedDict

import torch


def named_params(spec, flat_values):
    """Split a 1-D tensor of values into the model's named parameters (canonical order, align 1)."""
    H, hd = spec["hidden"], spec["head_dim"]
    shapes = OrderedDict()
    shapes["embed"] = (spec["vocab"], H)
    for l in range(spec["n_layers"]):
        p = f"layers.{l}."
        shapes[p + "in_norm"] = (H,)
        shapes[p + "q"] = (spec["n_q_heads"] * hd, H)
        shapes[p + "k"] = (spec["n_kv_heads"] * hd, H)
        shapes[p + "v"] = (spec["n_kv_heads"] * hd, H)
        if spec["qk_norm"]:
            shapes[p + "q_norm"] = (hd,)
            shapes[p + "k_norm"] = (hd,)
        shapes[p + "o"] = (H, spec["n_q_heads"] * hd)
        shapes[p + "post_norm"] = (H,)
        if spec["n_experts"] == 0:
            shapes[p + "gate"] = (spec["ffn"], H)
            shapes[p + "up"] = (spec["ffn"], H)
            shapes[p + "down"] = (H, spec["ffn"])
        else:
            shapes[p + "router"] = (spec["n_experts"], H)
            for e in range(spec["n_experts"]):
                q = p + f"experts.{e}."
                shapes[q + "gate"] = (spec["moe_ffn"], H)
                shapes[q + "up"] = (spec["moe_ffn"], H)
                shapes[q + "down"] = (H, spec["moe_ffn"])
    shapes["final_norm"] = (H,)
    if not spec["tied"]:
        shapes["lm_head"] = (spec["vocab"], H)
    sizes = [int(torch.Size(s).numel()) for s in shapes.values()]
    assert sum(sizes) == flat_values.numel()
    pieces = torch.split(flat_values, sizes)
    return OrderedDict((n, t.view(s)) for (n, s), t in zip(shapes.items(), pieces))


def _vocab_rows(w, tp, t, pad_to, fill):
    """Rows of rank t after padding the vocabulary up to a multiple of pad_to (padding rows = fill)."""
    if pad_to:
        extra = -w.shape[0] % pad_to
        w = torch.nn.functional.pad(w, (0, 0, 0, extra), value=fill)
    return w.chunk(tp, dim=0)[t]


def rollout_state(spec, params, tp, t, kv_replicate=False, vocab_pad=0, moe_tp=1, moe_ep=1, moe_ep_rank=0, fill=-1):
    """Fused, tensor-parallel-sliced rollout tensors for rank t of tp (values untouched; vocabulary
    padding rows hold `fill`)."""
    out = OrderedDict()
    nkv = spec["n_kv_heads"]

    def kv(w):
        if kv_replicate and tp > nkv:  # one head per rank, each head on tp / nkv consecutive ranks
            return w.view(nkv, spec["head_dim"], -1)[t // (tp // nkv)]
        return w.chunk(tp, dim=0)[t]

    out["embed"] = _vocab_rows(params["embed"], tp, t, vocab_pad, fill)
    for l in range(spec["n_layers"]):
        p = f"layers.{l}."
        out[p + "in_norm"] = params[p + "in_norm"]
        out[p + "qkv"] = torch.cat([params[p + "q"].chunk(tp, dim=0)[t], kv(params[p + "k"]), kv(params[p + "v"])], dim=0)
        if spec["qk_norm"]:
            out[p + "q_norm"] = params[p + "q_norm"]
            out[p + "k_norm"] = params[p + "k_norm"]
        out[p + "o"] = params[p + "o"].chunk(tp, dim=1)[t]
        out[p + "post_norm"] = params[p + "post_norm"]
        if spec["n_experts"] == 0:
            out[p + "gate_up"] = torch.cat([params[p + n].chunk(tp, dim=0)[t] for n in ("gate", "up")], dim=0)
            out[p + "down"] = params[p + "down"].chunk(tp, dim=1)[t]
        else:
            out[p + "router"] = params[p + "router"]
            E = spec["n_experts"]
            mine = list(torch.arange(E).chunk(moe_ep)[moe_ep_rank])  # expert parallelism: a contiguous block
            mt, mr = (tp, t) if moe_tp > 1 else (1, 0)                # expert tensor parallelism
            out[p + "w13"] = torch.stack(
                [torch.cat([params[p + f"experts.{int(e)}.gate"].chunk(mt, dim=0)[mr],
                            params[p + f"experts.{int(e)}.up"].chunk(mt, dim=0)[mr]], dim=0) for e in mine])
            out[p + "w2"] = torch.stack([params[p + f"experts.{int(e)}.down"].chunk(mt, dim=1)[mr] for e in mine])
    out["final_norm"] = params["final_norm"]
    if not spec["tied"]:
        out["lm_head"] = _vocab_rows(params["lm_head"], tp, t, vocab_pad, fill)
    return out
