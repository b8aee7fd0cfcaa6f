"""Helpers shared by the GPU parity tests (not collected as tests)."""
import numpy as np
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

MAX_ABS = 1e-2       # tolerances of the parity bar: max-abs and relative Frobenius
REL_FRO = 5e-3


def to_items(x: torch.Tensor) -> np.ndarray:
    """[rows, heads, T, D] bf16 (any device) -> [rows*heads, T, D] float64 numpy."""
    r, h, t, d = x.shape
    return x.detach().to("cpu").to(torch.float64).reshape(r * h, t, d).numpy()


def check_close(got: torch.Tensor, want: np.ndarray, what: str, max_abs=MAX_ABS, rel_fro=REL_FRO):
    g = to_items(got) if got.dim() == 4 else got.detach().cpu().double().numpy()
    assert np.isfinite(g).all(), what + ": non-finite output"
    err = np.abs(g - want).max()
    fro = np.linalg.norm(g - want) / max(np.linalg.norm(want), 1e-300)
    assert err <= max_abs, "%s: max-abs %.3e > %.1e" % (what, err, max_abs)
    assert fro <= rel_fro, "%s: relative Frobenius %.3e > %.1e" % (what, fro, rel_fro)
    return err, fro


class Cache:
    """Thin test-side holder: creates a cache over a torch-owned arena."""

    def __init__(self, layers, heads, head_dim, rows, sides, policies, softmax_scale=0.0, own_arena=True, flags=0,
                 token_budgets=None):
        self.desc, self._keep = B.make_desc(layers, heads, head_dim, rows, sides, policies, softmax_scale, flags,
                                            token_budgets)
        self.arena = None
        if own_arena:
            n = B.amskv_cache_required_bytes(self.desc)
            self.arena = torch.empty(n, dtype=torch.uint8, device="cuda")
            self.h = B.amskv_cache_create(self.desc, self.arena, n)
        else:
            self.h = B.amskv_cache_create(self.desc)
        self.sides = tuple(sides)
        self.policies = list(policies)

    def close(self):
        if self.h:
            B.amskv_cache_destroy(self.h)
            self.h = None
            self.arena = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()


def tensor_path_available(head_dim=64) -> bool:
    if not torch.cuda.is_available():
        return False
    with Cache(1, 1, head_dim, 1, (1,), [(1, 1, False)]) as c:
        return B.lib.amskv_set_attend_path(c.h, B.PATH_TENSOR) == B.OK


def run_pass(cache: Cache, qkv, path=B.PATH_AUTO, layers=None, fused=False):
    """Appends and attends every scale; qkv[k] = (Q, K, V) device tensors.  Returns outs[layer][k].
    fused: through amskv_append_attend (True), or only at the scales listed."""
    B.amskv_cache_reset(cache.h)
    B.amskv_set_attend_path(cache.h, path)
    layers = range(len(cache.policies)) if layers is None else layers
    outs = {l: [] for l in layers}
    for k, (q, kk, v) in enumerate(qkv):
        for l in layers:
            o = torch.full_like(q, float("nan"))
            if fused is True or (fused and k in fused):
                B.amskv_append_attend(cache.h, l, k, kk, v, q, o)
            else:
                B.amskv_append(cache.h, l, k, kk, v)
                B.amskv_attend(cache.h, l, k, q, o)
            outs[l].append(o)
    torch.cuda.synchronize()
    assert B.amskv_status(cache.h) == 0
    return outs


def oracle_outputs(qkv, policy, scale, items=None):
    """Oracle result per scale for one layer policy; items = optional list of item indices."""
    c, w, dem = policy
    Ks = [to_items(k) for _, k, _ in qkv]
    Vs = [to_items(v) for _, _, v in qkv]
    if items is not None:
        Ks = [k[items] for k in Ks]
        Vs = [v[items] for v in Vs]
    outs = []
    for k, (q, _, _) in enumerate(qkv):
        Q = to_items(q)
        if items is not None:
            Q = Q[items]
        outs.append(oracle.attend_selected(Q, Ks, Vs, oracle.keep_set(k, c, w, dem), scale))
    return outs


def make_qkv(rows, heads, sides, head_dim, seed, device="cuda", peaked=False):
    gen = synth.peaked_qkv_for_scale if peaked else synth.qkv_for_scale
    return [gen(rows, heads, s * s, head_dim, seed, k, device) for k, s in enumerate(sides)]
