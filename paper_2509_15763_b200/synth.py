"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds no arithmetic of the method: it only names the workloads and
draws random tensors.  Everything is produced in the INTERLEAVED token order
(one gist after every ``r`` raw tokens), on the CPU, from
``torch.Generator().manual_seed(seed)``; tensors are drawn in the order
Q, K, V, dO as float32 normal samples and rounded to bfloat16
(round-to-nearest-even), so the CUDA path and the fp64 CPU check read
bit-identical values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

BASE_SEED = 20250915
PAGE = 64  # tokens per cache block


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    raw_len: int      # T
    ratio: int        # r
    window: int       # W, raw tokens
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    num_sinks: int = 0
    k_scale: float = 1.0
    v_scale: float = 1.0
    dout_scale: float = 1.0  # dO is drawn as N(0, 1) * dout_scale
    seed: int = BASE_SEED
    forward_only: bool = False  # the workload is a prefill: no backward pass

    @property
    def num_gists(self) -> int:
        return self.raw_len // self.ratio

    @property
    def total_len(self) -> int:
        return self.num_sinks + self.raw_len + self.num_gists

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark workloads.
WORKLOADS = {
    "tiny": Workload("tiny", 1, 448, 7, 64, 1, 1, 64, seed=BASE_SEED + 0),
    "llama8b_layer": Workload("llama8b_layer", 1, 16384, 8, 1024, 32, 8, 128,
                              k_scale=0.5, seed=BASE_SEED + 1),
    "train_batch": Workload("train_batch", 4, 32768, 4, 2048, 32, 8, 128, seed=BASE_SEED + 2),
    "long_prefill": Workload("long_prefill", 1, 131072, 16, 4096, 32, 8, 128, seed=BASE_SEED + 3,
                             forward_only=True),
}

# The shapes of the paper's own speed table (appendix): one attention layer, batch 1, 32 heads (MHA),
# head_dim 128, 16K to 128K raw tokens, ratio 4 or 8, with the main experiments' 128 sinks and
# 128-token window.  Context for the numbers the paper prints, not one of the five workloads above.
for _i, _ctx in enumerate((16, 32, 64, 128)):
    for _r in (4, 8):
        _name = f"table4_{_ctx}k_r{_r}"
        WORKLOADS[_name] = Workload(_name, 1, _ctx * 1024, _r, 128, 32, 32, 128, num_sinks=128,
                                    seed=BASE_SEED + 10 + 2 * _i + (_r == 8))

    # the table's "causal attention" row: plain causal attention over the same raw tokens, which is the
    # method's own special case of a single gist unit (ratio = window = T, one gist at the very end, no sinks)
    _name = f"table4_{_ctx}k_causal"
    WORKLOADS[_name] = Workload(_name, 1, _ctx * 1024, _ctx * 1024, _ctx * 1024, 32, 32, 128, seed=BASE_SEED + 30 + _i)


@dataclass(frozen=True)
class DecodeWorkload:
    name: str
    num_seqs: int
    num_gists: int
    window_raw: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    seed: int = BASE_SEED + 4

    @property
    def seq_len(self) -> int:
        return self.num_gists + self.window_raw


DECODE_WORKLOADS = {
    "decode_cache": DecodeWorkload("decode_cache", 64, 8192, 1024, 32, 8, 128),
}


def attention_inputs(w: Workload, with_grad: bool = True, dout_fp32: bool = False):
    """-> dict of interleaved tensors: q [B,N,Hq,D], k, v [B,N,Hkv,D] (bf16), dout."""
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    N = w.total_len

    def draw(h):
        return torch.randn(w.batch, N, h, w.head_dim, generator=g, dtype=torch.float32)

    q = draw(w.num_q_heads).to(torch.bfloat16)
    k = (draw(w.num_kv_heads) * w.k_scale).to(torch.bfloat16)
    v = (draw(w.num_kv_heads) * w.v_scale).to(torch.bfloat16)
    out = {"q": q, "k": k, "v": v}
    if with_grad:
        d = draw(w.num_q_heads) * w.dout_scale
        out["dout"] = d if dout_fp32 else d.to(torch.bfloat16)
    return out


def decode_inputs(w: DecodeWorkload, spare_blocks: int = 0):
    """Paged compressed cache: k_cache, v_cache [num_blocks, Hkv, PAGE, D] bf16,
    block_table [S, blocks_per_seq] int32 (a seeded random permutation of the
    physical block ids), seq_lens [S] int32, q [S, Hq, D] bf16."""
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    per_seq = -(-w.seq_len // PAGE)
    nb = w.num_seqs * per_seq + spare_blocks
    q = torch.randn(w.num_seqs, w.num_q_heads, w.head_dim, generator=g).to(torch.bfloat16)
    kc = torch.randn(nb, w.num_kv_heads, PAGE, w.head_dim, generator=g).to(torch.bfloat16)
    vc = torch.randn(nb, w.num_kv_heads, PAGE, w.head_dim, generator=g).to(torch.bfloat16)
    perm = torch.randperm(nb, generator=g)[: w.num_seqs * per_seq].to(torch.int32)
    table = perm.reshape(w.num_seqs, per_seq).contiguous()
    lens = torch.full((w.num_seqs,), w.seq_len, dtype=torch.int32)
    return {"q": q, "k_cache": kc, "v_cache": vc, "block_table": table, "seq_lens": lens}
