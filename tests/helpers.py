"""Glue shared by the parity tests: feeds the same seeded inputs to the oracle and to the CUDA path."""
from __future__ import annotations

import numpy as np
import torch

from oracle import verillm_oracle as vo
from paper_2509_24257_b200 import synth


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 bit patterns (numpy has no bf16)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_model(wl: synth.Workload, n_layers=None, tokens=None) -> vo.Model:
    """Oracle model of a workload.  The oracle keeps the fp32 master weights when the workload says so,
    else the bf16 values the GPU gets.  With `tokens`, only the embedding rows in use are generated."""
    shape = wl.shape
    L = shape.n_layers if n_layers is None else n_layers
    f32 = wl.oracle_weights == "f32"
    dt = torch.float32 if f32 else torch.bfloat16
    conv = (lambda t: t.numpy()) if f32 else bits
    layers = [{k: conv(v) for k, v in synth.layer_weights(wl, l, "cpu", dt).items()} for l in range(L)]
    final = conv(synth.final_norm_weights(wl, "cpu", dt))
    if tokens is None:
        embed, rows = conv(synth.embed_weights(wl, "cpu", dt)), None
    else:
        ids = sorted(set(int(t) for t in np.asarray(tokens).reshape(-1)))
        embed = conv(synth.embed_weights(wl, "cpu", dt, rows=torch.tensor(ids)))
        rows = {t: i for i, t in enumerate(ids)}
    import dataclasses
    return vo.make_model(dataclasses.replace(shape, n_layers=L), embed, final, layers, rows)


def oracle_committed(m: vo.Model, tokens: np.ndarray, check_seq, check_pos, precision="bf16") -> np.ndarray:
    """Prover trace from the oracle's own token-by-token decode: [n_layers, n_check, d] float64 (not yet
    rounded to the commit dtype).  Each sequence is decoded only as far as its last checked position."""
    out = np.zeros((m.n_layers, len(check_seq), m.d_model))
    for b in range(tokens.shape[0]):
        sel = np.nonzero(np.asarray(check_seq) == b)[0]
        if sel.size == 0:
            continue
        upto = int(np.max(np.asarray(check_pos)[sel])) + 1
        st = vo.forward_decode_kvcache(m, tokens[b, :upto], precision)
        for s in sel:
            out[:, s] = st[:, int(check_pos[s])]
    return out


def oracle_tol(**kw) -> vo.Tol:
    return vo.Tol(**kw)


def rel_l2(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Row-wise ||a-b|| / ||b|| over the last axis."""
    return np.linalg.norm(a - b, axis=-1) / np.maximum(np.linalg.norm(b, axis=-1), 1e-30)


class LazyLayers:
    """Sequence of per-layer float64 weight dicts of a workload, one layer materialised per access.
    `device` is where the seeded generator runs (the values are identical on any device)."""

    def __init__(self, wl: synth.Workload, n_layers: int, device="cpu"):
        self.wl, self.n, self.device = wl, n_layers, device

    def __len__(self):
        return self.n

    def __getitem__(self, l: int):
        lw = synth.layer_weights(self.wl, l, self.device, torch.bfloat16)
        return {k: vo.as_f64(bits(v)) for k, v in lw.items()}


def oracle_model_streamed(wl: synth.Workload, tokens, device="cpu") -> vo.Model:
    """Oracle model whose layers are generated on access and whose embedding holds only the rows in use."""
    s = wl.shape
    ids = sorted(set(int(t) for t in np.asarray(tokens).reshape(-1)))
    embed = vo.as_f64(bits(synth.embed_weights(wl, device, torch.bfloat16, rows=torch.tensor(ids))))
    final = vo.as_f64(bits(synth.final_norm_weights(wl, "cpu", torch.bfloat16)))
    return vo.Model(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab,
                    float(s.rope_base), float(s.rms_eps), embed, final, LazyLayers(wl, s.n_layers, device),
                    {t: i for i, t in enumerate(ids)})


def gpu_model(wl: synth.Workload, max_checks: int, device="cuda:0"):
    """Library handle holding the workload's weights, generated on the device layer by layer."""
    from paper_2509_24257_b200 import binding as vb

    m = vb.Model(wl.shape, wl.n_tokens, max_checks, wl.batch, device)
    m.load_globals(synth.embed_weights(wl, device), synth.final_norm_weights(wl, device))
    for l in range(wl.shape.n_layers):
        m.load_layer(l, synth.layer_weights(wl, l, device))
    return m
