"""Seeded synthetic inputs for the DAF prefill-attention path.

This module holds input generation only: a counter-based random generator and
the five workload shapes.  It contains none of the method's arithmetic and is
the one module that both the CUDA path's callers and the CPU oracle's callers
use, so that both sides always see the same tensors.

The paper evaluates on public long-context RAG suites with Qwen2.5-7B weights
(Experimental Setup paragraph).  Neither is available offline; these inputs
take only the *shapes* of those workloads (contexts of 1k-32k tokens made of
documents of a few hundred tokens, a short question, the attention geometry of
Qwen2.5-7B / Llama-3-8B / Qwen2.5-14B) and stand in for them.

Generator: element i of tensor `tid` of layer `layer` of config `cfg` is
    splitmix64(seed(cfg, layer, tid) + i-th counter) -> uniform(0,1) (53 bits)
two uniforms per normal draw through Box-Muller, evaluated in float64, then
rounded to the storage type.  All integer steps are exact on any device.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, Dict, Iterator, List, Optional, Tuple

import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_BASE_SEED = 0xDAF0260721599

TENSOR_IDS = {"q_fresh": 0, "k_fresh": 1, "v_fresh": 2, "k_cached": 3, "v_cached": 4,
              "scores": 5, "idx_perm": 6, "hot_docs": 7}


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit integer as a signed one (torch has no uint64 arithmetic)."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def splitmix64_int(x: int) -> int:
    """splitmix64 finaliser on a Python integer (host-side seeds and small draws)."""
    z = (x + _GOLDEN) & _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def splitmix64_tensor(counter: torch.Tensor, seed: int) -> torch.Tensor:
    """splitmix64 of (seed + counter) on an int64 tensor; wraps modulo 2**64."""
    z = counter + _s64(seed) + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def tensor_seed(config_id: int, layer: int, tensor_id: int) -> int:
    return splitmix64_int(_BASE_SEED ^ (config_id << 40) ^ (layer << 16) ^ tensor_id)


def uniform01(n: int, seed: int, device="cpu", start: int = 0) -> torch.Tensor:
    """n float64 uniforms in [0, 1) from counters start .. start+n-1."""
    c = torch.arange(start, start + n, dtype=torch.int64, device=device)
    bits = _lsr(splitmix64_tensor(c, seed), 11)
    return bits.to(torch.float64) * (1.0 / (1 << 53))


def standard_normal(n: int, seed: int, device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """n float64 N(0,1) draws (Box-Muller, cosine branch; counters 2i and 2i+1 feed draw i)."""
    out = torch.empty(n, dtype=torch.float64, device=device)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        u = uniform01(2 * m, seed, device, start=2 * lo).view(m, 2)
        rad = torch.sqrt(-2.0 * torch.log1p(-u[:, 0]))
        out[lo:lo + m] = rad * torch.cos((2.0 * math.pi) * u[:, 1])
    return out


def normal_bf16(shape: Tuple[int, ...], seed: int, device="cpu") -> torch.Tensor:
    n = 1
    for s in shape:
        n *= s
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    chunk = 1 << 24
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        u = uniform01(2 * m, seed, device, start=2 * lo).view(m, 2)
        rad = torch.sqrt(-2.0 * torch.log1p(-u[:, 0]))
        out[lo:lo + m] = (rad * torch.cos((2.0 * math.pi) * u[:, 1])).to(torch.bfloat16)
    return out.view(*shape)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One workload shape.  `selection` is how the important tokens are chosen:
    'given' (a seeded random index set is passed in), 'lognormal' or
    'pareto_clustered' (importance scores are drawn and the top k are selected)."""
    name: str
    config_id: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    layers: int
    L_d: int
    doc_len: int
    L_q: int
    r: float
    selection: str
    n_sig: int = 1
    k: int = -1     # number of important tokens; stated for the named configurations, otherwise supplied by
                    # the caller through with_k() (the counting rule belongs to the library and to the oracle)

    @property
    def N(self) -> int:
        return self.L_d + self.L_q

    @property
    def n_docs(self) -> int:
        return self.L_d // self.doc_len

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    def with_k(self, num_important: Callable[[int, float], int]) -> "Workload":
        """The same workload with k filled in by `num_important(L_d, r)` (the library's or the oracle's)."""
        return self if self.k >= 0 else dataclasses.replace(self, k=int(num_important(self.L_d, self.r)))


CONFIGS: Dict[str, Workload] = {
    "c0": Workload("c0", 0, 28, 4, 128, 1, 1024, 256, 32, 0.15, "given", k=154),
    "c1": Workload("c1", 1, 28, 4, 128, 28, 6144, 512, 64, 0.15, "lognormal", k=922),
    "c2": Workload("c2", 2, 32, 8, 128, 32, 16384, 512, 128, 0.10, "lognormal", k=1639),
    "c3": Workload("c3", 3, 28, 4, 128, 28, 32768, 512, 128, 0.20, "pareto_clustered", k=6554),
}


# Beyond the five stated configurations: the shape of the paper's longest evaluation point (a 136k-token
# context with r = 0.3, Table 1), four layers of it.  Used by the benchmark and one sampled parity test.
EXTRA_CONFIGS: Dict[str, Workload] = {
    "x136k": Workload("x136k", 5, 28, 4, 128, 4, 139264, 512, 128, 0.30, "lognormal", k=41780),
}


def sweep_points(num_important: Optional[Callable[[int, float], int]] = None) -> List[Workload]:
    """The single-layer sweep on the Qwen2.5-14B attention shape.  k is filled in when the caller hands over
    the counting function (the library's or the oracle's)."""
    pts = []
    for L_d in (2048, 8192, 16384, 32768):
        for r in (0.05, 0.10, 0.20, 0.30):
            w = Workload(f"c4_L{L_d}_r{r:.2f}", 4, 40, 8, 128, 1, L_d, 512, 128, r, "lognormal")
            pts.append(w.with_k(num_important) if num_important is not None else w)
    return pts


def tiny(name: str = "tiny", L_d: int = 48, doc_len: int = 16, L_q: int = 5, r: float = 0.25,
         n_q_heads: int = 4, n_kv_heads: int = 2, head_dim: int = 8, selection: str = "lognormal",
         n_sig: int = 3, config_id: int = 99, num_important: Optional[Callable[[int, float], int]] = None) -> Workload:
    """A small shape for brute-force checks."""
    w = Workload(name, config_id, n_q_heads, n_kv_heads, head_dim, 1, L_d, doc_len, L_q, r, selection, n_sig)
    return w.with_k(num_important) if num_important is not None else w


def given_indices(w: Workload, layer: int = 0) -> torch.Tensor:
    """k distinct positions: the first k entries of a seeded Fisher-Yates shuffle of 0..L_d-1, sorted."""
    if w.k < 0:
        raise ValueError("workload without a count of important tokens: use with_k()")
    seed = tensor_seed(w.config_id, layer, TENSOR_IDS["idx_perm"])
    perm = list(range(w.L_d))
    for i in range(w.L_d - 1, 0, -1):
        j = splitmix64_int(seed + i) % (i + 1)
        perm[i], perm[j] = perm[j], perm[i]
    return torch.tensor(sorted(perm[: w.k]), dtype=torch.int32)


def importance_scores(w: Workload, layer: int = 0, device="cpu") -> torch.Tensor:
    """fp32 [n_sig, L_d] importance scores for the score-driven workloads."""
    seed = tensor_seed(w.config_id, layer, TENSOR_IDS["scores"])
    n = w.n_sig * w.L_d
    if w.selection == "lognormal":
        s = torch.exp(standard_normal(n, seed, device))
    elif w.selection == "pareto_clustered":
        alpha = 1.5
        u = uniform01(n, seed, device)
        s = torch.pow(1.0 - u, -1.0 / alpha)
        n_hot = max(1, int(math.ceil(0.2 * w.n_docs)))
        n_cold = w.n_docs - n_hot
        boost = (7.0 * n_cold / (3.0 * n_hot)) ** (1.0 / alpha) if n_cold > 0 else 1.0
        hseed = tensor_seed(w.config_id, layer, TENSOR_IDS["hot_docs"])
        docs = list(range(w.n_docs))
        for i in range(w.n_docs - 1, 0, -1):
            j = splitmix64_int(hseed + i) % (i + 1)
            docs[i], docs[j] = docs[j], docs[i]
        mult = torch.ones(w.n_docs, dtype=torch.float64, device=device)
        mult[torch.tensor(sorted(docs[:n_hot]), device=device)] = boost
        s = (s.view(w.n_sig, w.n_docs, w.doc_len) * mult.view(1, w.n_docs, 1)).reshape(-1)
    else:
        raise ValueError(f"workload {w.name} has no score-driven selection")
    return s.to(torch.float32).view(w.n_sig, w.L_d)


def make_layer(w: Workload, layer: int = 0, device="cpu") -> Dict[str, Optional[torch.Tensor]]:
    """All inputs of one layer: fresh Q/K/V over N = L_d + L_q rows, the offline
    (cached) document K/V, and either importance scores or a given index set.
    Token-major bf16, every element an independent N(0,1) draw."""
    sd = lambda t: tensor_seed(w.config_id, layer, TENSOR_IDS[t])  # noqa: E731
    D = w.head_dim
    out: Dict[str, Optional[torch.Tensor]] = {
        "q_fresh": normal_bf16((w.N, w.n_q_heads, D), sd("q_fresh"), device),
        "k_fresh": normal_bf16((w.N, w.n_kv_heads, D), sd("k_fresh"), device),
        "v_fresh": normal_bf16((w.N, w.n_kv_heads, D), sd("v_fresh"), device),
        "k_cached": normal_bf16((w.L_d, w.n_kv_heads, D), sd("k_cached"), device),
        "v_cached": normal_bf16((w.L_d, w.n_kv_heads, D), sd("v_cached"), device),
        "scores": None,
        "idx_in": None,
    }
    if w.selection == "given":
        out["idx_in"] = given_indices(w, layer).to(device)
    else:
        out["scores"] = importance_scores(w, layer, device)
    return out


def iter_layers(w: Workload, device="cpu") -> Iterator[Dict[str, Optional[torch.Tensor]]]:
    for layer in range(w.layers):
        yield make_layer(w, layer, device)


def attention_pairs(w: Workload) -> Dict[str, int]:
    """Visible (query, key) pairs of each stage; 4 * head_dim * n_q_heads flop per pair."""
    k, L_q, L_d, N = w.k, w.L_q, w.L_d, w.N
    if k < 0:
        raise ValueError("workload without a count of important tokens: use with_k()")
    return {
        "important": k * (k + 1) // 2,
        "question": L_q * L_d + L_q * (L_q + 1) // 2,
        "full": N * (N + 1) // 2,
    }


def attention_flops(w: Workload) -> Dict[str, float]:
    per_pair = 4.0 * w.head_dim * w.n_q_heads
    return {name: per_pair * n for name, n in attention_pairs(w).items()}
