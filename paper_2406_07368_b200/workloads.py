"""Seeded synthetic inputs for the linear-attention layer.

This module only draws random numbers, rounds them to the storage type and
builds draft-token trees.  It contains none of the layer's arithmetic, so both
the CUDA path and an independent checker can be fed from it.

All floating-point arrays are returned as numpy float32 whose values are
exactly representable in the storage type named by ``io`` ("f32" or "bf16").
Every draw comes from a counter-based generator (Philox) keyed by
``(seed, stream)``, so a draw never depends on the order in which other draws
were made.

Shapes follow the layer's conventions: q, k, v are [B, H, T, d] (prefill),
[B, H, d] (one decode token) or [B, H, N, d] (a draft tree of N nodes);
the depthwise convolution weights are [H, d, W] with tap 0 multiplying the
current token; a tree is a parent array [B, N] with -1 for children of the
committed prefix and parent[n] < n.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# Stream identifiers: one Philox key per kind of draw.
_STREAM_QKV = 1
_STREAM_W = 2
_STREAM_DECODE = 3
_STREAM_TREE = 4
_STREAM_DRAFT = 5
_STREAM_ACCEPT = 6
_STREAM_STATE = 7
_STREAM_TOKENS = 8
_STREAM_PROMPT = 9


def rng(seed: int, stream: int, a: int = 0, b: int = 0) -> np.random.Generator:
    """Generator keyed by (seed, stream, a, b); independent of call order."""
    key0 = (int(seed) & 0xFFFFFFFF) | ((int(stream) & 0xFFFFFFFF) << 32)
    key1 = (int(a) & 0xFFFFFFFF) | ((int(b) & 0xFFFFFFFF) << 32)
    return np.random.Generator(np.random.Philox(key=[key0, key1]))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even), kept as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def store(x: np.ndarray, io: str) -> np.ndarray:
    """Round to the storage type: "bf16" or "f32"."""
    if io == "bf16":
        return round_to_bf16(x)
    if io == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(f"unknown io type {io!r}")


def gaussian(gen: np.random.Generator, shape, scale: float, io: str) -> np.ndarray:
    x = gen.standard_normal(size=shape, dtype=np.float32) * np.float32(scale)
    return store(x, io)


def qkv(seed: int, shape, scale: float, io: str, stream: int = _STREAM_QKV, a: int = 0, v_mean: float = 0.0):
    """Three independent Gaussian tensors of the same shape.  `v_mean` shifts the values v: with a non-zero mean the
    attention term (a weighted mean of values) keeps its size at late positions instead of averaging out."""
    q, k, v = (gaussian(rng(seed, stream, a, i), shape, scale, io) for i in range(3))
    if v_mean != 0.0:
        v = store(v + np.float32(v_mean), io)
    return q, k, v


def conv_weights(seed: int, H: int, d: int, W: int) -> np.ndarray:
    """Depthwise taps ~ N(0, 1/W) as float32 [H, d, W] (variance 1/3 at W = 3)."""
    g = rng(seed, _STREAM_W)
    return (g.standard_normal(size=(H, d, W), dtype=np.float32) * np.float32(W ** -0.5)).astype(np.float32)


# --------------------------------------------------------------------------
# Draft trees
# --------------------------------------------------------------------------

def random_tree(gen: np.random.Generator, N: int, max_depth: int = 5, max_fanout: int = 4) -> np.ndarray:
    """Parent array of a random draft tree built by sequential attachment.

    Node n picks its parent uniformly among the committed prefix (-1, while it
    has fewer than ``max_fanout`` children) and the earlier nodes that are
    shallower than ``max_depth`` and have fewer than ``max_fanout`` children.
    Depth counts from 1 at a child of the prefix.
    """
    parent = np.full(N, -1, dtype=np.int32)
    depth = np.zeros(N, dtype=np.int32)
    nchild = np.zeros(N, dtype=np.int32)
    root_children = 0
    for n in range(N):
        cands = []
        if root_children < max_fanout:
            cands.append(-1)
        for m in range(n):
            if depth[m] < max_depth and nchild[m] < max_fanout:
                cands.append(m)
        if not cands:
            raise ValueError("tree is full: N too large for max_depth/max_fanout")
        p = cands[int(gen.integers(len(cands)))]
        parent[n] = p
        if p < 0:
            root_children += 1
            depth[n] = 1
        else:
            nchild[p] += 1
            depth[n] = depth[p] + 1
    return parent


def chain_tree(N: int) -> np.ndarray:
    return np.arange(-1, N - 1, dtype=np.int32)


def tree_depths(parent: np.ndarray) -> np.ndarray:
    depth = np.zeros(len(parent), dtype=np.int32)
    for n, p in enumerate(parent):
        depth[n] = 1 if p < 0 else depth[p] + 1
    return depth


def random_accept(gen: np.random.Generator, parent: np.ndarray) -> int:
    """Deepest accepted node: a uniform leaf, then a uniform prefix length of its path."""
    N = len(parent)
    has_child = np.zeros(N, dtype=bool)
    for p in parent:
        if p >= 0:
            has_child[p] = True
    leaves = np.nonzero(~has_child)[0]
    leaf = int(leaves[int(gen.integers(len(leaves)))])
    path = []
    n = leaf
    while n >= 0:
        path.append(n)
        n = int(parent[n])
    path.reverse()
    L = int(gen.integers(1, len(path) + 1))
    return path[L - 1]


def token_batch(seed: int, rnd: int, B: int, N: int, vocab: int = 4):
    """Token ids for the acceptance step: what the drafter proposed at every node and what the verifier predicts
    after the prefix and after every node.  A small vocabulary makes matches (and so accepted chains of several
    tokens) frequent.  Returns (draft_token [B,N], pred_root [B], pred [B,N]) int32."""
    g = rng(seed, _STREAM_TOKENS, rnd)
    draft = g.integers(0, vocab, size=(B, N), dtype=np.int32)
    pred_root = g.integers(0, vocab, size=(B,), dtype=np.int32)
    pred = g.integers(0, vocab, size=(B, N), dtype=np.int32)
    return draft, pred_root, pred


def tree_batch(seed: int, rnd: int, B: int, N: int, max_depth: int = 5, max_fanout: int = 4):
    """Per-sequence trees and accepted nodes for one speculative round."""
    parent = np.stack([random_tree(rng(seed, _STREAM_TREE, rnd, b), N, max_depth, max_fanout)
                       for b in range(B)]).astype(np.int32)
    accept = np.array([random_accept(rng(seed, _STREAM_ACCEPT, rnd, b), parent[b]) for b in range(B)],
                      dtype=np.int32)
    return parent, accept


# --------------------------------------------------------------------------
# The workload shapes
# --------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    io: str            # "f32" | "bf16"
    B: int
    H: int
    d: int
    T: int             # prefill length
    W: int             # live causal taps of the depthwise convolution
    chunk: int
    phi: str           # "elu1" | "relu"
    eps: float
    seed: int
    scale: float       # standard deviation of q, k, v
    decode_steps: int = 0
    tree_nodes: int = 0
    max_depth: int = 5
    rounds: int = 0
    extra: dict = field(default_factory=dict)

    def weights(self) -> np.ndarray:
        return conv_weights(self.seed, self.H, self.d, self.W)

    def prefill_inputs(self, B: int | None = None, H: int | None = None, T: int | None = None):
        """q, k, v [B, H, T, d]; sub-sampling B/H/T draws a smaller tensor of the same law."""
        shape = (B or self.B, H or self.H, T or self.T, self.d)
        return qkv(self.seed, shape, self.scale, self.io)

    def prompt_of_sequence(self, b: int, T: int | None = None):
        """q, k, v [1, H, T, d] of sequence b alone, keyed by b: for batches whose prompts are too large to draw as
        one array, the prompt is built sequence by sequence."""
        return qkv(self.seed, (1, self.H, T or self.T, self.d), self.scale, self.io, stream=_STREAM_PROMPT, a=b)

    def decode_inputs(self, step: int, B: int | None = None, H: int | None = None):
        shape = (B or self.B, H or self.H, self.d)
        return qkv(self.seed, shape, self.extra.get("decode_scale", self.scale), self.io,
                   stream=_STREAM_DECODE, a=step)

    def draft_inputs(self, rnd: int, B: int | None = None, H: int | None = None):
        shape = (B or self.B, H or self.H, self.tree_nodes, self.d)
        return qkv(self.seed, shape, self.extra.get("decode_scale", self.scale), self.io,
                   stream=_STREAM_DRAFT, a=rnd)

    def trees(self, rnd: int, B: int | None = None):
        return tree_batch(self.seed, rnd, B or self.B, self.tree_nodes, self.max_depth)


def tiny_fp32() -> Workload:
    """B=1, H=2, d=64, T=256 fp32, elu+1, 3 taps; 16 decode steps; 4-node chain, accept 2."""
    return Workload("tiny_fp32", "f32", 1, 2, 64, 256, 3, 64, "elu1", 0.0, 0, 1.0,
                    decode_steps=16, tree_nodes=4, rounds=1,
                    extra={"chain": True, "accept_node": 1})


def llama7b_prefill() -> Workload:
    """B=4, H=32, d=128, T=2048 bf16, chunk 64, elu+1, 3 taps; inputs N(0,1)/sqrt(d)."""
    return Workload("llama7b_prefill", "bf16", 4, 32, 128, 2048, 3, 64, "elu1", 0.0, 1, 128 ** -0.5)


def batched_decode() -> Workload:
    """64 sequences, H=32, d=128: 2048-token N(0,1) bf16 prefill, then 1024 decode steps."""
    return Workload("batched_decode", "bf16", 64, 32, 128, 2048, 3, 64, "elu1", 0.0, 2, 1.0,
                    decode_steps=1024)


def tree_verify() -> Workload:
    """16 sequences, H=32, d=128: 1024-token prefill; 64-node trees, depth <= 5; 256 rounds."""
    return Workload("tree_verify", "bf16", 16, 32, 128, 1024, 3, 64, "elu1", 0.0, 3, 1.0,
                    tree_nodes=64, max_depth=5, rounds=256)


def long_prefill() -> Workload:
    """B=1, H=32, d=128, T=32768 bf16, chunk 128, ReLU, eps 1e-6, 5 taps; then 512 decode steps."""
    return Workload("long_prefill", "bf16", 1, 32, 128, 32768, 5, 128, "relu", 1e-6, 4, 128 ** -0.5,
                    decode_steps=512)


def prompt_gen() -> Workload:
    """One sequence, H=32, d=128, bf16, elu+1, 3 taps: a prompt of P tokens is prefilled and G tokens are then
    generated one by one, for the (P, G) pairs of the paper's table of inference latency at various prefill and
    decode sizes: (340, 160), (60, 20), (7000, 200), (1700, 400).  Inputs N(0,1)."""
    return Workload("prompt_gen", "bf16", 1, 32, 128, 7000, 3, 64, "elu1", 0.0, 5, 1.0,
                    extra={"shapes": [(340, 160), (60, 20), (7000, 200), (1700, 400)]})


def grouped_block() -> Workload:
    """The three-branch block on the LLaMA-2-7B-shaped prefill: B=4, H=32, d=128, T=2048 bf16, groups of 64 (the
    paper's group size for LLaMA), softmax scale 1/sqrt(d), alpha 1, elu+1, 3 taps; inputs N(0,1)/sqrt(d)."""
    return Workload("grouped_block", "bf16", 4, 32, 128, 2048, 3, 64, "elu1", 0.0, 6, 128 ** -0.5,
                    extra={"alpha": 1.0, "softmax_scale": 128 ** -0.5})


def prefill_taps32() -> Workload:
    """The LLaMA-2-7B-shaped prefill with the longest tap window: 32 live taps, which is what a convolution kernel of
    63 (the paper's choice for FLASH) keeps under the causal mask."""
    return Workload("prefill_taps32", "bf16", 4, 32, 128, 2048, 32, 64, "elu1", 0.0, 7, 128 ** -0.5)


def tree_verify_taps8() -> Workload:
    """The tree_verify shapes with 8 live taps: twice as many as the tensor cores gather."""
    return Workload("tree_verify_taps8", "bf16", 16, 32, 128, 1024, 8, 64, "elu1", 0.0, 8, 1.0,
                    tree_nodes=64, max_depth=5, rounds=256)


WORKLOADS = {w().name: w for w in (tiny_fp32, llama7b_prefill, batched_decode, tree_verify, long_prefill, prompt_gen,
                                   grouped_block, prefill_taps32, tree_verify_taps8)}
