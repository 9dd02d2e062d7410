"""Seeded synthetic inputs for the verifier-prefill path.

This module only *generates inputs*: model shapes, random-init weights, token
streams, the sampled check positions and the tampering recipes.  It holds none
of the verifier's arithmetic (no transformer forward, no comparison, no
verdict) and imports neither the CUDA binding nor the CPU oracle, so both can
be fed from it.

Every value is a pure function of (seed, tensor id, element index): a
splitmix64-style integer mix picks one of 65536 equiprobable quantiles of the
normal distribution from a table.  Only wrapping 64-bit integer operations and
a table gather are involved, so the same tensor is produced bit for bit on the
CPU and on a CUDA device, one tensor (or one layer) at a time, without ever
materialising the whole model on the host.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Iterable, List, Optional, Tuple

import numpy as np
import torch

# --------------------------------------------------------------------------- shapes


@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Llama-style decoder shape (pre-norm, RMSNorm, RoPE, GQA, SwiGLU, no biases)."""

    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def d_q(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim

    def gemm_flops_per_token(self) -> float:
        d, f = self.d_model, self.d_ffn
        return 2.0 * self.n_layers * (d * (self.d_q + 2 * self.d_kv) + self.d_q * d + 3 * d * f)

    def attn_flops_per_token(self, seq_len: int) -> float:
        """Causal attention counted as half the square (QK^T and PV)."""
        return self.n_layers * 4.0 * self.n_heads * self.head_dim * (seq_len + 1) / 2.0

    def n_params(self) -> int:
        d, f = self.d_model, self.d_ffn
        per_layer = d * (self.d_q + 2 * self.d_kv) + self.d_q * d + 3 * d * f + 2 * d
        return self.vocab * d + self.n_layers * per_layer + d


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic verification job: a model shape plus a batch of served sequences."""

    name: str
    shape: ModelShape
    batch: int
    prompt_len: int
    gen_len: int
    check_frac: float
    seed: int
    oracle_weights: str = "bf16"  # "f32": the oracle keeps the fp32 master values
    token_seed_offset: int = 0  # replicas of one model draw different sequences, checks and tampering

    @property
    def seq_len(self) -> int:
        return self.prompt_len + self.gen_len

    @property
    def n_tokens(self) -> int:
        return self.batch * self.seq_len

    @property
    def n_check(self) -> int:
        return max(1, int(round(self.check_frac * self.n_tokens)))

    def total_flops(self) -> float:
        s = self.shape
        return self.n_tokens * (s.gemm_flops_per_token() + s.attn_flops_per_token(self.seq_len))

    def with_layers(self, n_layers: int) -> "Workload":
        """Same widths and batch, reduced depth (weights of the first layers are unchanged)."""
        return dataclasses.replace(
            self, name=f"{self.name}-L{n_layers}", shape=dataclasses.replace(self.shape, n_layers=n_layers)
        )

    def with_batch(self, batch: int, prompt_len: int, gen_len: int) -> "Workload":
        return dataclasses.replace(
            self, name=f"{self.name}-b{batch}x{prompt_len + gen_len}", batch=batch, prompt_len=prompt_len, gen_len=gen_len
        )


_BASE_SEED = 20250924

WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload(
        "tiny", ModelShape(1, 256, 4, 4, 64, 768, 1024, 10000.0), 1, 32, 32, 1.0, _BASE_SEED + 1, "f32"
    ),
    "small": Workload(
        "small", ModelShape(4, 1024, 16, 4, 64, 2816, 32000, 10000.0), 4, 256, 256, 0.01, _BASE_SEED + 2
    ),
    "llama8b": Workload(
        "llama8b", ModelShape(32, 4096, 32, 8, 128, 14336, 128256, 500000.0), 8, 512, 512, 0.01, _BASE_SEED + 3
    ),
    "llama8b_long": Workload(
        "llama8b_long", ModelShape(32, 4096, 32, 8, 128, 14336, 128256, 500000.0), 2, 2048, 2048, 0.005,
        _BASE_SEED + 4,
    ),
    "llama70b": Workload(
        "llama70b", ModelShape(80, 8192, 64, 8, 128, 28672, 128256, 500000.0), 1, 1024, 1024, 0.01, _BASE_SEED + 5
    ),
}

# --------------------------------------------------------------------------- generator

_GOLDEN = -7046029254386353131  # 0x9E3779B97F4A7C15 as a signed 64-bit integer
_MUL1 = -4658895280553007687  # 0xBF58476D1CE4E5B9
_MUL2 = -7723592293110705685  # 0x94D049BB133111EB
_TABLE_BITS = 16


def _wrap64(x: int) -> int:
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_scalar(x: int) -> int:
    """splitmix64 finaliser on Python integers (used for per-tensor keys)."""
    m = (1 << 64) - 1
    x = (x + 0x9E3779B97F4A7C15) & m
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & m
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & m
    x = x ^ (x >> 31)
    return x


def _lsr_(z: torch.Tensor, k: int, tmp: torch.Tensor) -> torch.Tensor:
    """tmp <- logical (z >> k) for int64 tensors (arithmetic shift, then mask)."""
    torch.bitwise_right_shift(z, k, out=tmp)
    tmp.bitwise_and_((1 << (64 - k)) - 1)
    return tmp


def _mix_range(key: int, start: int, n: int, device: torch.device) -> torch.Tensor:
    """64-bit mixed values for element indices start .. start+n-1 (int64 tensor, wrapping)."""
    z = torch.arange(start, start + n, dtype=torch.int64, device=device)
    tmp = torch.empty_like(z)
    z.mul_(_GOLDEN).add_(_wrap64(key))
    z.bitwise_xor_(_lsr_(z, 30, tmp)).mul_(_MUL1)
    z.bitwise_xor_(_lsr_(z, 27, tmp)).mul_(_MUL2)
    z.bitwise_xor_(_lsr_(z, 31, tmp))
    return z


_quantiles_f32: Optional[torch.Tensor] = None


def normal_quantile_table() -> torch.Tensor:
    """65536 equiprobable standard-normal quantiles, fp32, on the CPU."""
    global _quantiles_f32
    if _quantiles_f32 is None:
        from scipy.special import ndtri

        n = 1 << _TABLE_BITS
        q = ndtri((np.arange(n, dtype=np.float64) + 0.5) / n)
        _quantiles_f32 = torch.from_numpy(q.astype(np.float32))
    return _quantiles_f32


def _tensor_key(seed: int, uid: int) -> int:
    return _mix_scalar((seed & ((1 << 64) - 1)) ^ _mix_scalar(uid))


def normal_tensor(
    seed: int,
    uid: int,
    shape: Tuple[int, ...],
    std: float,
    mean: float = 0.0,
    device: torch.device | str = "cpu",
    dtype: torch.dtype = torch.bfloat16,
) -> torch.Tensor:
    """Tensor of `mean + std * N(0,1)` values: fp32 master values, cast (RNE) to `dtype`.

    The fp32 master of an element is identical whichever dtype is requested, so the
    bf16 tensor is exactly the round-to-nearest-even image of the fp32 one.
    """
    device = torch.device(device)
    numel = int(math.prod(shape))
    key = _tensor_key(seed, uid)
    table = (normal_quantile_table() * np.float32(std) + np.float32(mean)).to(device)
    table = table.to(dtype)
    out = torch.empty(numel, dtype=dtype, device=device)
    chunk = (1 << 25) if device.type == "cuda" else (1 << 20)
    for s in range(0, numel, chunk):
        n = min(chunk, numel - s)
        z = _mix_range(key, s, n, device)
        z.bitwise_and_((1 << _TABLE_BITS) - 1)
        out[s : s + n] = table[z]
    return out.view(*shape)


# tensor kinds inside a layer (uid = 16 * (layer + 1) + kind; layer -1 holds the globals)
_KINDS = {
    "attn_norm": 0, "wq": 1, "wk": 2, "wv": 3, "wo": 4, "ffn_norm": 5, "w_gate": 6, "w_up": 7, "w_down": 8,
}
_WEIGHT_STD = 0.02
_GAMMA_STD = 0.1  # norm gains are 1 + 0.1 * N(0,1): a dropped or misplaced gain must show up in parity


def weight_std(shape: ModelShape) -> float:
    """Std of the projection weights: 0.02 at d_model = 256, carried to wider models at constant gain
    std * sqrt(d_model) = 0.32.  (A plain 0.02 at d_model = 4096 has gain 1.28 per projection: such a
    random network amplifies rounding noise from layer to layer, unlike the trained models it stands for.)"""
    return _WEIGHT_STD * math.sqrt(256.0 / max(shape.d_model, 256))


def layer_tensor_shapes(shape: ModelShape) -> Dict[str, Tuple[int, ...]]:
    """Shapes of one layer's tensors; every projection is [out_features, in_features] row-major."""
    d, f = shape.d_model, shape.d_ffn
    return {
        "attn_norm": (d,), "wq": (shape.d_q, d), "wk": (shape.d_kv, d), "wv": (shape.d_kv, d),
        "wo": (d, shape.d_q), "ffn_norm": (d,), "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
    }


def layer_weights(
    wl: Workload, layer: int, device: torch.device | str = "cpu", dtype: torch.dtype = torch.bfloat16
) -> Dict[str, torch.Tensor]:
    out = {}
    for name, shp in layer_tensor_shapes(wl.shape).items():
        uid = 16 * (layer + 1) + _KINDS[name]
        if name.endswith("norm"):
            out[name] = normal_tensor(wl.seed, uid, shp, _GAMMA_STD, 1.0, device, dtype)
        else:
            out[name] = normal_tensor(wl.seed, uid, shp, weight_std(wl.shape), 0.0, device, dtype)
    return out


def embed_weights(
    wl: Workload, device: torch.device | str = "cpu", dtype: torch.dtype = torch.bfloat16,
    rows: Optional[torch.Tensor] = None,
) -> torch.Tensor:
    """Embedding table [vocab, d_model]; with `rows` only those rows are generated ([len(rows), d_model])."""
    s = wl.shape
    if rows is None:
        return normal_tensor(wl.seed, 1, (s.vocab, s.d_model), _WEIGHT_STD, 0.0, device, dtype)
    device = torch.device(device)
    key = _tensor_key(wl.seed, 1)
    table = (normal_quantile_table() * np.float32(_WEIGHT_STD)).to(device).to(dtype)
    rows = rows.to(device=device, dtype=torch.int64).reshape(-1)
    out = torch.empty(rows.numel(), s.d_model, dtype=dtype, device=device)
    for i, r in enumerate(rows.tolist()):
        z = _mix_range(key, r * s.d_model, s.d_model, device)
        z.bitwise_and_((1 << _TABLE_BITS) - 1)
        out[i] = table[z]
    return out


def final_norm_weights(
    wl: Workload, device: torch.device | str = "cpu", dtype: torch.dtype = torch.bfloat16
) -> torch.Tensor:
    return normal_tensor(wl.seed, 2, (wl.shape.d_model,), _GAMMA_STD, 1.0, device, dtype)


def lm_head_weights(
    wl: Workload, device: torch.device | str = "cpu", dtype: torch.dtype = torch.bfloat16
) -> torch.Tensor:
    """Output head [vocab, d_model] (untied from the embedding)."""
    s = wl.shape
    return normal_tensor(wl.seed, 3, (s.vocab, s.d_model), weight_std(s), 0.0, device, dtype)


def model_weights(
    wl: Workload, device: torch.device | str = "cpu", dtype: torch.dtype = torch.bfloat16
) -> Dict[str, object]:
    """All tensors of the model: {'embed', 'final_norm', 'layers': [dict per layer]}."""
    return {
        "embed": embed_weights(wl, device, dtype),
        "final_norm": final_norm_weights(wl, device, dtype),
        "layers": [layer_weights(wl, l, device, dtype) for l in range(wl.shape.n_layers)],
    }


def fake_quantise(w: torch.Tensor, bits: int = 8) -> torch.Tensor:
    """Weights of a prover that serves a quantised model (the quantisation attack): every output row is
    rounded to a symmetric `bits`-bit integer grid spanning its largest magnitude, and widened back to the
    tensor's dtype.  Input recipe of the attack traces only; the verifier never sees these weights."""
    w32 = w.to(torch.float32)
    qmax = float(2 ** (bits - 1) - 1)
    scale = w32.abs().amax(dim=-1, keepdim=True).clamp_min(1e-30) / qmax
    return (torch.round(w32 / scale).clamp_(-qmax, qmax) * scale).to(w.dtype)


def quantised_model_weights(weights: Dict[str, object], bits: int = 8) -> Dict[str, object]:
    """The same model with every projection matrix fake-quantised (norm gains and the embedding untouched)."""
    layers = [{k: (v if k.endswith("norm") else fake_quantise(v, bits)) for k, v in lw.items()} for lw in weights["layers"]]
    return {"embed": weights["embed"], "final_norm": weights["final_norm"], "layers": layers}


# --------------------------------------------------------------------------- sequences


def token_streams(wl: Workload) -> np.ndarray:
    """int32 [batch, prompt_len + gen_len] tokens, uniform over the vocabulary."""
    n = wl.n_tokens
    z = _mix_range(_tensor_key(wl.seed + 1 + wl.token_seed_offset, 0), 0, n, torch.device("cpu"))
    z = torch.bitwise_right_shift(z, 1).bitwise_and_((1 << 62) - 1)
    tok = torch.remainder(z, wl.shape.vocab).to(torch.int32)
    return tok.view(wl.batch, wl.seq_len).numpy().copy()


def cu_seqlens(wl: Workload) -> np.ndarray:
    return (np.arange(wl.batch + 1, dtype=np.int64) * wl.seq_len).astype(np.int32)


def check_positions(wl: Workload, n_check: Optional[int] = None, force: Iterable[Tuple[int, int]] = ()) -> Tuple[np.ndarray, np.ndarray]:
    """Sampled (sequence, position) pairs, uniform without replacement over all batch*seq_len
    positions (prompt and generated alike), in draw order (unsorted).  `force` pairs are
    placed first (the tampering recipes need their position in the check set)."""
    n = wl.n_check if n_check is None else n_check
    rng = np.random.Generator(np.random.PCG64(wl.seed + 2 + wl.token_seed_offset))
    flat = rng.choice(wl.n_tokens, size=min(n, wl.n_tokens), replace=False)
    forced = [s * wl.seq_len + p for s, p in force]
    if forced:
        rest = [x for x in flat.tolist() if x not in set(forced)]
        flat = np.array((forced + rest)[: max(n, len(forced))], dtype=np.int64)
    return (flat // wl.seq_len).astype(np.int32), (flat % wl.seq_len).astype(np.int32)


# --------------------------------------------------------------------------- tampering


def tamper_rng(wl: Workload) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(wl.seed + 3 + wl.token_seed_offset))


def swap_token(tokens: np.ndarray, seq: int, pos: int, vocab: int, rng: np.random.Generator) -> np.ndarray:
    """Copy of `tokens` with tokens[seq, pos] replaced by a different uniformly drawn token."""
    out = tokens.copy()
    new = int(rng.integers(0, vocab - 1))
    if new >= int(tokens[seq, pos]):
        new += 1
    out[seq, pos] = new
    return out


def add_state_noise(
    committed: np.ndarray, slots: Iterable[int], layers: Optional[Iterable[int]], scale: float,
    rng: np.random.Generator,
) -> np.ndarray:
    """Copy of committed states [n_layers, n_check, d_model] (float) with Gaussian noise of
    `scale` x (RMS of the vector it is added to) at the given check slots and layers
    (None = every layer).  The caller re-rounds to the commit dtype."""
    out = np.array(committed, dtype=np.float64, copy=True)
    n_layers = out.shape[0]
    for slot in slots:
        for l in range(n_layers) if layers is None else layers:
            v = out[l, slot]
            rms = float(np.sqrt(np.mean(v * v)))
            out[l, slot] = v + scale * rms * rng.standard_normal(v.shape[0])
    return out


def to_commit_dtype(states: np.ndarray, commit_dtype: str) -> torch.Tensor:
    """Round float states to the serialisation dtype of the trace ('bf16' or 'f32')."""
    t = torch.from_numpy(np.ascontiguousarray(states, dtype=np.float64))
    return t.to(torch.bfloat16 if commit_dtype == "bf16" else torch.float32)
