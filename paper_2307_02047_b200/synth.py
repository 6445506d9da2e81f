"""Seeded synthetic workloads for the CAME optimizer step.

This module only *describes* parameter sets (tensor shapes) and *draws* their
initial values and per-step gradients.  It contains none of the optimizer's
arithmetic: it is the one piece of code that both the CUDA path's tests and the
CPU oracle's tests may use, so that both sides are fed bit-identical inputs.

Every draw is keyed by ``(seed, tensor index, step)`` through numpy's Philox
counter-based bit generator, so any tensor of any step can be regenerated alone
and in any order.

Gradients are returned either as ``float32`` arrays or, for the bf16 workloads,
as ``uint16`` arrays holding bfloat16 bit patterns (round-to-nearest-even from
float32).  ``widen()`` turns either into float64 exactly.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple

import numpy as np

F32 = "f32"
BF16 = "bf16"

_PARAM_STEP_KEY = (1 << 32) - 1   # "step" slot used for the parameter draw
_SIGMA_STEP_KEY = (1 << 32) - 2   # "step" slot used for the per-tensor sigma draw
_ROWS_STREAM = 1 << 40            # added to the tensor index for row-mask draws


@dataclasses.dataclass(frozen=True)
class TensorSpec:
    """One parameter tensor: a matrix (rows x cols, row-major) or a vector."""
    name: str
    rows: int
    cols: int          # 1 for vectors
    ndim: int          # 1 or 2

    @property
    def numel(self) -> int:
        return self.rows * self.cols

    @property
    def shape(self) -> Tuple[int, ...]:
        return (self.rows,) if self.ndim == 1 else (self.rows, self.cols)


@dataclasses.dataclass(frozen=True)
class Workload:
    """A named parameter set plus its gradient recipe and hyper-parameters."""
    name: str
    tensors: Tuple[TensorSpec, ...]
    grad_dtype: str            # F32 or BF16
    grad_kind: str             # "normal_fixed", "normal_loguniform", "student_t3"
    grad_scale: float          # sigma for normal_fixed / scale for student_t3
    zero_row_frac: float       # fraction of gradient rows zeroed each step
    zero_row_tensors: Tuple[int, ...]   # tensor indices the row mask applies to
    steps: int
    hparams: dict

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)


def mat(name: str, rows: int, cols: int) -> TensorSpec:
    return TensorSpec(name, int(rows), int(cols), 2)


def vec(name: str, n: int) -> TensorSpec:
    return TensorSpec(name, int(n), 1, 1)


PAPER_HPARAMS = dict(lr=2e-4, beta1=0.9, beta2=0.999, beta3=0.9999,
                     eps1=1e-30, eps2=1e-16, clip_d=1.0, weight_decay=0.0)


def _bert_like(hidden: int, ffn: int, layers: int, vocab: int, pos: int) -> List[TensorSpec]:
    ts = [mat("tok_emb", vocab, hidden), mat("pos_emb", pos, hidden)]
    for l in range(layers):
        p = f"l{l}."
        ts += [mat(p + n, hidden, hidden) for n in ("wq", "wk", "wv", "wo")]
        ts += [mat(p + "w_in", hidden, ffn), mat(p + "w_out", ffn, hidden)]
        ts += [vec(p + n, hidden) for n in ("bq", "bk", "bv", "bo")]
        ts += [vec(p + "b_in", ffn), vec(p + "b_out", hidden)]
        ts += [vec(p + n, hidden) for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b")]
    return ts


def _gpt2_like(hidden: int, ffn: int, layers: int, vocab: int, pos: int) -> List[TensorSpec]:
    ts = [mat("tok_emb", vocab, hidden), mat("pos_emb", pos, hidden)]
    for l in range(layers):
        p = f"l{l}."
        ts += [mat(p + "w_qkv", hidden, 3 * hidden), mat(p + "w_proj", hidden, hidden),
               mat(p + "w_in", hidden, ffn), mat(p + "w_out", ffn, hidden)]
        ts += [vec(p + "b_qkv", 3 * hidden), vec(p + "b_proj", hidden),
               vec(p + "b_in", ffn), vec(p + "b_out", hidden)]
        ts += [vec(p + n, hidden) for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b")]
    return ts


def _llama_like(hidden: int, ffn: int, layers: int, vocab: int) -> List[TensorSpec]:
    ts = [mat("tok_emb", vocab, hidden)]
    for l in range(layers):
        p = f"l{l}."
        ts += [mat(p + n, hidden, hidden) for n in ("wq", "wk", "wv", "wo")]
        ts += [mat(p + "w_gate", hidden, ffn), mat(p + "w_up", hidden, ffn),
               mat(p + "w_down", ffn, hidden)]
        ts += [vec(p + "norm1", hidden), vec(p + "norm2", hidden)]
    ts += [vec("norm_f", hidden), mat("lm_head", vocab, hidden)]
    return ts


def workload(name: str) -> Workload:
    """Return one of the named synthetic workloads.

    ``toy``          one 512x256 fp32 matrix and one 256 bias, 10 steps
    ``bert_base``    BERT-base-shaped set, fp32 gradients, per-tensor sigma
    ``bert_large``   BERT-large-shaped set, bf16 gradients, 20% embedding rows zeroed
    ``gpt2_medium``  GPT-2-medium-shaped set, bf16 heavy-tailed gradients, weight decay
    ``llama7b``      LLaMA-7B-shaped set, bf16 gradients of sigma 1e-3
    ``llama7b_layer`` the seven matrices and two vectors of one llama7b layer
    ``mat:RxC[:bf16]`` a single matrix of the shape/scale sweep
    """
    hp = dict(PAPER_HPARAMS)
    if name == "toy":
        return Workload(name, (mat("w", 512, 256), vec("b", 256)), F32, "normal_fixed",
                        1e-3, 0.0, (), 10, hp)
    if name == "bert_base":
        return Workload(name, tuple(_bert_like(768, 3072, 12, 30522, 512)), F32,
                        "normal_loguniform", 0.0, 0.0, (), 100, hp)
    if name == "bert_large":
        return Workload(name, tuple(_bert_like(1024, 4096, 24, 30522, 512)), BF16,
                        "normal_loguniform", 0.0, 0.2, (0, 1), 50, hp)
    if name == "gpt2_medium":
        hp["weight_decay"] = 0.01
        return Workload(name, tuple(_gpt2_like(1024, 4096, 24, 50257, 1024)), BF16,
                        "student_t3", 1e-3, 0.0, (), 20, hp)
    if name == "llama7b":
        return Workload(name, tuple(_llama_like(4096, 11008, 32, 32000)), BF16,
                        "normal_fixed", 1e-3, 0.0, (), 5, hp)
    if name == "llama7b_layer":
        full = _llama_like(4096, 11008, 1, 32000)
        return Workload(name, tuple(full[1:10]), BF16, "normal_fixed", 1e-3, 0.0, (), 5, hp)
    if name.startswith("mat:"):
        parts = name.split(":")
        r, c = parts[1].lower().split("x")
        dt = BF16 if len(parts) > 2 and parts[2] == "bf16" else F32
        return Workload(name, (mat("w", int(r), int(c)),), dt, "normal_fixed", 1e-3,
                        0.0, (), 5, hp)
    raise KeyError(f"unknown workload {name!r}")


SWEEP_SHAPES = ((1024, 1024), (2048, 2048), (4096, 4096), (8192, 8192), (16384, 16384),
                (1, 65536), (65536, 1), (128256, 4096))


def with_zero_rows_everywhere(w: Workload, frac: float = 0.2) -> Workload:
    """Variant that zeroes a fresh subset of rows in EVERY matrix each step."""
    idx = tuple(i for i, t in enumerate(w.tensors) if t.ndim == 2)
    return dataclasses.replace(w, name=w.name + "+zero_rows", zero_row_frac=frac,
                               zero_row_tensors=idx)


# ----------------------------------------------------------------------------
# draws
# ----------------------------------------------------------------------------

def _rng(seed: int, stream: int, step: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1),
                                                     ((int(stream) << 32) | int(step)) & (2**64 - 1)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def widen(a: np.ndarray) -> np.ndarray:
    """Exact float64 value of a float32 array or of a uint16 array of bf16 bit patterns."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


def make_param(w: Workload, seed: int, i: int) -> np.ndarray:
    """Initial value of parameter tensor ``i``, float32, N(0, 0.02^2)."""
    t = w.tensors[i]
    z = _rng(seed, i, _PARAM_STEP_KEY).standard_normal(t.numel, dtype=np.float32)
    return (z * np.float32(0.02)).reshape(t.shape)


def make_params(w: Workload, seed: int) -> List[np.ndarray]:
    """Initial parameters of every tensor (see make_param)."""
    return [make_param(w, seed, i) for i in range(len(w.tensors))]


def tensor_sigma(w: Workload, seed: int, i: int) -> float:
    """Per-tensor gradient scale: fixed, or log-uniform in [1e-5, 1e-2] drawn once per tensor."""
    if w.grad_kind == "normal_loguniform":
        u = _rng(seed, i, _SIGMA_STEP_KEY).random()
        return float(10.0 ** (-5.0 + 3.0 * u))
    return float(w.grad_scale)


def make_grad(w: Workload, seed: int, i: int, step: int) -> np.ndarray:
    """Gradient of tensor ``i`` at ``step`` (1-based): float32 array or uint16 bf16 bits."""
    t = w.tensors[i]
    rng = _rng(seed, i, step)
    s = np.float32(tensor_sigma(w, seed, i))
    if w.grad_kind == "student_t3":
        z = rng.standard_normal(t.numel, dtype=np.float32)
        q = np.zeros(t.numel, dtype=np.float32)
        for _ in range(3):
            n = rng.standard_normal(t.numel, dtype=np.float32)
            q += n * n
        g = s * z / np.sqrt(q / np.float32(3.0))
    else:
        g = s * rng.standard_normal(t.numel, dtype=np.float32)
    g = g.reshape(t.shape)
    if w.zero_row_frac > 0.0 and i in w.zero_row_tensors and t.ndim == 2:
        mask = _rng(seed, _ROWS_STREAM + i, step).random(t.rows) < w.zero_row_frac
        g[mask, :] = np.float32(0.0)
    if w.grad_dtype == BF16:
        return f32_to_bf16_bits(g)
    return g.astype(np.float32, copy=False)


def make_grads(w: Workload, seed: int, step: int, indices: Sequence[int] | None = None,
               workers: int = 0) -> List[np.ndarray]:
    """All (or the listed) gradients of one step.  Draws are keyed per tensor, so generating
    them on ``workers`` threads gives the same bits as generating them one by one."""
    idx = list(range(len(w.tensors)) if indices is None else indices)
    if workers > 1 and len(idx) > 1:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=workers) as ex:
            return list(ex.map(lambda i: make_grad(w, seed, i, step), idx))
    return [make_grad(w, seed, i, step) for i in idx]


def rank1_sign_matrix(rows: int, cols: int, seed: int, step: int = 1
                      ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """A float64 matrix whose element-wise square is exactly rank one.

    Returns ``(g, a, b)`` with ``g[i, j] = s[i, j] * sqrt(a[i] * b[j])`` for random
    signs ``s`` and positive vectors ``a`` (rows) and ``b`` (cols) that do NOT
    depend on ``step`` (only the signs do), so the same ``a, b`` recur across steps.
    """
    ab = _rng(seed, 7, 0)
    a = ab.uniform(0.5, 2.0, rows)
    b = ab.uniform(0.5, 2.0, cols) * 1e-6
    sgn = np.where(_rng(seed, 8, step).random((rows, cols)) < 0.5, -1.0, 1.0)
    g = sgn * np.sqrt(np.outer(a, b))
    return g, a, b
