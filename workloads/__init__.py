"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This module only *generates inputs*: tensor contents, request lengths, block tables,
checkpoint indices and schedules.  It holds none of the movement arithmetic (no pool or
packed-buffer address formula, no descriptor) and imports neither the oracle nor the CUDA
package, so both sides receive exactly the same arrays.

Contents are counter based: element i of a buffer filled with seed s is a pure function
of (s, i), evaluated identically by numpy on the host and by torch integer ops on the
device, so multi-GB device buffers never need a host mirror and the oracle can look up any
sampled source element on its own.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

SEED_BASE = 260806007 * 10  # config k uses SEED_BASE + k

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


# --------------------------------------------------------------------------------------
# counter-based contents
# --------------------------------------------------------------------------------------
def _mix64_np(seed: int, idx: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser of (idx * golden + seed * C2), on uint64 arrays."""
    with np.errstate(over="ignore"):
        z = idx.astype(np.uint64) * np.uint64(_GOLDEN) + np.uint64((seed * _C2) & _M64)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_C1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_C2)
        z = z ^ (z >> np.uint64(31))
    return z


def _s64(v: int) -> int:
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix64_torch(seed: int, idx):
    """Same function as _mix64_np on int64 torch tensors (two's-complement wraparound)."""
    def lsr(x, k):
        return (x >> k) & ((1 << (64 - k)) - 1)
    z = idx * _s64(_GOLDEN) + _s64(seed * _C2)
    z = (z ^ lsr(z, 30)) * _s64(_C1)
    z = (z ^ lsr(z, 27)) * _s64(_C2)
    return z ^ lsr(z, 31)


_NORMAL_SCALE = np.float32(0.02 / math.sqrt(4.0 * (65536.0 ** 2 - 1.0) / 12.0))


def bits16_np(seed: int, start: int, count: int) -> np.ndarray:
    """Uniform random 16-bit patterns: elements [start, start+count) as uint16."""
    idx = np.arange(start, start + count, dtype=np.uint64)
    return (_mix64_np(seed, idx) & np.uint64(0xFFFF)).astype(np.uint16)


def bits16_at_np(seed: int, idx) -> np.ndarray:
    """Uniform 16-bit patterns at arbitrary element indices."""
    return (_mix64_np(seed, np.asarray(idx, dtype=np.uint64)) & np.uint64(0xFFFF)).astype(np.uint16)


def normal_bf16_at_np(seed: int, idx) -> np.ndarray:
    """bf16 bit patterns of approximately N(0, 0.02) values at element indices idx.

    The value is an Irwin-Hall sum of the hash's four 16-bit fields, centred, scaled in
    float32 and rounded to nearest-even bf16: integer and single-multiply arithmetic only,
    so host and device agree bit for bit.
    """
    z = _mix64_np(seed, np.asarray(idx, dtype=np.uint64))
    m = np.uint64(0xFFFF)
    s = ((z & m) + ((z >> np.uint64(16)) & m) + ((z >> np.uint64(32)) & m) + (z >> np.uint64(48))).astype(np.int64)
    f = (s - 131070).astype(np.float32) * _NORMAL_SCALE
    u = f.view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def normal_bf16_np(seed: int, start: int, count: int) -> np.ndarray:
    return normal_bf16_at_np(seed, np.arange(start, start + count, dtype=np.uint64))


def fill_np(buf_u8: np.ndarray, seed: int, kind: str = "bits16", chunk: int = 1 << 22) -> None:
    """Fill a flat uint8 array (even length) with 16-bit elements of the given kind."""
    v = buf_u8.view(np.uint16)
    fn = bits16_np if kind == "bits16" else normal_bf16_np
    for s in range(0, v.size, chunk):
        n = min(chunk, v.size - s)
        v[s:s + n] = fn(seed, s, n)


def fill_torch(buf_u8, seed: int, kind: str = "bits16", chunk: int = 1 << 26) -> None:
    """Fill a flat uint8 torch tensor (any device, even length) with the same elements as fill_np."""
    import torch
    v = buf_u8.view(torch.int16)
    n_el = v.numel()
    for s in range(0, n_el, chunk):
        n = min(chunk, n_el - s)
        idx = torch.arange(s, s + n, dtype=torch.int64, device=buf_u8.device)
        z = _mix64_torch(seed, idx)
        if kind == "bits16":
            v[s:s + n] = (z & 0xFFFF).to(torch.int16)
        else:
            tot = (z & 0xFFFF) + ((z >> 16) & 0xFFFF) + ((z >> 32) & 0xFFFF) + ((z >> 48) & 0xFFFF)
            f = (tot - 131070).to(torch.float32) * float(_NORMAL_SCALE)
            v[s:s + n] = f.to(torch.bfloat16).view(torch.int16)


# --------------------------------------------------------------------------------------
# samplers
# --------------------------------------------------------------------------------------
def lognormal_lengths(rng: np.random.Generator, n: int, mu: float, sigma: float,
                      lo: int, hi: int) -> np.ndarray:
    """round(exp(mu + sigma*N(0,1))) clipped to [lo, hi] (same family as the paper's Table 3)."""
    x = np.exp(mu + sigma * rng.standard_normal(n))
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def clipped_geometric(rng: np.random.Generator, n: int, p: float, hi: int) -> np.ndarray:
    """min(Geom(p) on {1,2,...}, hi)."""
    return np.minimum(rng.geometric(p, n), hi).astype(np.int64)


# --------------------------------------------------------------------------------------
# KV workloads
# --------------------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class KVShape:
    L: int
    B: int
    H: int
    D: int
    E: int = 2

    @property
    def tuple(self):
        return (self.L, self.B, self.H, self.D, self.E)

    @property
    def chunk_bytes(self):  # one block of one (layer, K|V) plane
        return self.B * self.H * self.D * self.E

    @property
    def block_bytes(self):  # one block over all layers, K and V
        return self.L * 2 * self.chunk_bytes

    @property
    def token_bytes(self):
        return self.L * 2 * self.H * self.D * self.E


LLAMA3_8B_KV = KVShape(L=32, B=16, H=8, D=128, E=2)
LLAMA3_70B_KV = KVShape(L=80, B=32, H=8, D=128, E=2)


@dataclasses.dataclass
class KVRequests:
    """R requests: valid tokens T[r] and a CSR block table (bt_off[R+1], bt[...])."""
    T: np.ndarray
    bt_off: np.ndarray
    bt: np.ndarray

    @property
    def n_blocks(self):
        return int(self.bt_off[-1])


def _csr(T: np.ndarray, B: int) -> np.ndarray:
    n = (np.asarray(T, dtype=np.int64) + B - 1) // B
    return np.concatenate([[0], np.cumsum(n)]).astype(np.int64)


def config1(seed: int = SEED_BASE + 1):
    """Correctness case: 1 layer, 64-block pool, 4 requests of 37/100/5/200 tokens."""
    shape = KVShape(L=1, B=16, H=8, D=128, E=2)
    NB = 64
    T = np.array([37, 100, 5, 200], dtype=np.int64)
    off = _csr(T, shape.B)
    rng_src, rng_dst = [np.random.default_rng(s) for s in np.random.SeedSequence(seed).spawn(2)]
    src = KVRequests(T, off, rng_src.permutation(NB)[:off[-1]].astype(np.int32))
    dst = KVRequests(T, off, rng_dst.permutation(NB)[:off[-1]].astype(np.int32))
    return shape, NB, src, dst


def admit_waves(n_blocks_per_req: np.ndarray, capacity: int):
    """Requests admitted in index order while the wave's block count stays <= capacity."""
    waves, cur, used = [], [], 0
    for r, n in enumerate(n_blocks_per_req):
        n = int(n)
        if n > capacity:
            raise ValueError(f"request {r} needs {n} blocks > wave capacity {capacity}")
        if used + n > capacity and cur:
            waves.append(np.array(cur, dtype=np.int64))
            cur, used = [], 0
        cur.append(r)
        used += n
    if cur:
        waves.append(np.array(cur, dtype=np.int64))
    return waves


def config2(NB: int = 20000, R: int = 256, wave_blocks: int | None = None,
            shape: KVShape = LLAMA3_8B_KV, seed: int = SEED_BASE + 2,
            median: int = 2048, sigma: float = 1.0, max_len: int = 32768, NB_dst: int | None = None):
    """Offload/reload waves: log-normal context lengths, fragmented block tables.

    Returns (shape, NB, T_all, waves); every wave is (src, dst): the table the wave's
    requests occupy when packed, and an independent fresh allocation (drawn from a pool of
    NB_dst blocks, default NB) they are reloaded into.
    """
    ss = np.random.SeedSequence(seed).spawn(3)
    T_all = lognormal_lengths(np.random.default_rng(ss[0]), R, math.log(median), sigma, 1, max_len)
    n_all = (T_all + shape.B - 1) // shape.B
    NB_dst = NB if NB_dst is None else NB_dst
    cap = min(NB, NB_dst) if wave_blocks is None else min(NB, NB_dst, wave_blocks)
    # a request larger than the wave capacity is truncated to it (recorded in T_all)
    too_big = n_all > cap
    T_all = np.where(too_big, cap * shape.B, T_all)
    rng_a, rng_b = np.random.default_rng(ss[1]), np.random.default_rng(ss[2])
    waves = []
    for ids in admit_waves((T_all + shape.B - 1) // shape.B, cap):
        T = T_all[ids]
        off = _csr(T, shape.B)
        src = KVRequests(T, off, rng_a.permutation(NB)[:off[-1]].astype(np.int32))
        dst = KVRequests(T, off, rng_b.permutation(NB_dst)[:off[-1]].astype(np.int32))
        waves.append((src, dst))
    return shape, NB, T_all, waves


def config4(NB: int = 4096, R: int = 1024, shape: KVShape = LLAMA3_70B_KV,
            seed: int = SEED_BASE + 4, lo: int = 512, hi: int = 8192, max_waves: int | None = None):
    """Pool-to-pool migration waves: uniform lengths, independent src and dst permutations."""
    ss = np.random.SeedSequence(seed).spawn(3)
    T_all = np.random.default_rng(ss[0]).integers(lo, hi + 1, R).astype(np.int64)
    rng_a, rng_b = np.random.default_rng(ss[1]), np.random.default_rng(ss[2])
    waves = []
    for ids in admit_waves((T_all + shape.B - 1) // shape.B, NB):
        T = T_all[ids]
        off = _csr(T, shape.B)
        src = KVRequests(T, off, rng_a.permutation(NB)[:off[-1]].astype(np.int32))
        dst = KVRequests(T, off, rng_b.permutation(NB)[:off[-1]].astype(np.int32))
        waves.append((src, dst))
        if max_waves is not None and len(waves) >= max_waves:
            break
    return shape, NB, T_all, waves


@dataclasses.dataclass
class MixedStep:
    """One scheduler step of the prefix-reload burst: block-granular, full blocks only."""
    reload_T: np.ndarray        # tokens per session (= blocks * B)
    reload_off: np.ndarray
    reload_host: np.ndarray     # source block ids in the host pool
    reload_dev: np.ndarray      # destination block ids in the device pool
    offload_T: np.ndarray
    offload_off: np.ndarray
    offload_dev: np.ndarray     # source block ids in the device pool
    offload_host: np.ndarray    # destination block ids in the host pool


def config5(NB_dev: int = 20000, NB_host: int = 262144, sessions: int = 512, steps: int = 200,
            shape: KVShape = LLAMA3_8B_KV, seed: int = SEED_BASE + 5, p: float = 1.0 / 12.0,
            max_prefix: int = 64, max_new: int = 4):
    """Generator of MixedStep: every session reloads min(Geom(p), 64) blocks from the host
    pool into scattered device blocks and offloads 1..4 device blocks into host blocks that
    are disjoint from the step's reload sources.  Device blocks are recycled each step."""
    rng = np.random.default_rng(seed)
    for _ in range(steps):
        k = clipped_geometric(rng, sessions, p, max_prefix)
        m = rng.integers(1, max_new + 1, sessions).astype(np.int64)
        host = rng.permutation(NB_host)[:int(k.sum() + m.sum())].astype(np.int32)
        dev = rng.permutation(NB_dev)[:int(k.sum() + m.sum())].astype(np.int32)
        nk = int(k.sum())
        yield MixedStep(
            reload_T=k * shape.B, reload_off=np.concatenate([[0], np.cumsum(k)]).astype(np.int64),
            reload_host=host[:nk], reload_dev=dev[:nk],
            offload_T=m * shape.B, offload_off=np.concatenate([[0], np.cumsum(m)]).astype(np.int64),
            offload_dev=dev[nk:], offload_host=host[nk:])


# --------------------------------------------------------------------------------------
# checkpoint workload
# --------------------------------------------------------------------------------------
@dataclasses.dataclass
class Checkpoint:
    """A flat blob's offset index: tensors back to back in `names` order, plus the
    tensor-parallel rule of each (split_dim -1 = replicated)."""
    names: list
    shapes: np.ndarray     # [N][4], unused leading... trailing dims are 1
    ndim: np.ndarray       # [N]
    E: np.ndarray          # [N] bytes per element
    byte_off: np.ndarray   # [N]
    split_dim: np.ndarray  # [N]
    nbytes_total: int

    @property
    def N(self):
        return len(self.names)

    def nbytes(self, i):
        return int(np.prod(self.shapes[i])) * int(self.E[i])


def llama_checkpoint(hidden=4096, layers=32, q_heads=32, kv_heads=8, head_dim=128, mlp=14336,
                     vocab=128256, E=2, pad_to: int = 1, order_seed: int | None = None,
                     lead_pad: int = 0) -> Checkpoint:
    """Llama-shaped state dict: embed, per layer [in_norm, q, k, v, o, post_norm, gate, up,
    down], final norm, lm_head; stored [out, in] row-major, tight (or padded to `pad_to`).
    Rules: q/k/v/gate/up/embed/lm_head split the output dim (0), o/down split the input dim
    (1), norms are replicated.  order_seed permutes the storage order; lead_pad shifts the
    whole blob (to exercise misaligned offsets)."""
    items = [("embed_tokens", (vocab, hidden), 0)]
    for l in range(layers):
        p = f"layers.{l}."
        items += [(p + "input_layernorm", (hidden,), -1),
                  (p + "q_proj", (q_heads * head_dim, hidden), 0),
                  (p + "k_proj", (kv_heads * head_dim, hidden), 0),
                  (p + "v_proj", (kv_heads * head_dim, hidden), 0),
                  (p + "o_proj", (hidden, q_heads * head_dim), 1),
                  (p + "post_attention_layernorm", (hidden,), -1),
                  (p + "gate_proj", (mlp, hidden), 0),
                  (p + "up_proj", (mlp, hidden), 0),
                  (p + "down_proj", (hidden, mlp), 1)]
    items += [("norm", (hidden,), -1), ("lm_head", (vocab, hidden), 0)]
    order = np.arange(len(items))
    if order_seed is not None:
        order = np.random.default_rng(order_seed).permutation(len(items))
    N = len(items)
    shapes = np.ones((N, 4), dtype=np.int64)
    ndim = np.zeros(N, dtype=np.int32)
    byte_off = np.zeros(N, dtype=np.int64)
    off = lead_pad
    for i in order:
        _, shp, _ = items[i]
        shapes[i, :len(shp)] = shp
        ndim[i] = len(shp)
        off = (off + pad_to - 1) // pad_to * pad_to if pad_to > 1 else off
        byte_off[i] = off
        off += int(np.prod(shp)) * E
    return Checkpoint(names=[it[0] for it in items], shapes=shapes, ndim=ndim,
                      E=np.full(N, E, dtype=np.int64), byte_off=byte_off,
                      split_dim=np.array([it[2] for it in items], dtype=np.int32),
                      nbytes_total=off)


def config3() -> Checkpoint:
    """The Llama-3-8B-shaped checkpoint: 291 bf16 tensors, 16 060 522 496 bytes."""
    return llama_checkpoint()


def shard_shape(ck: Checkpoint, i: int, world: int):
    s = [int(x) for x in ck.shapes[i]]
    if ck.split_dim[i] >= 0:
        s[ck.split_dim[i]] //= world
    return s


def moe_checkpoint(hidden=64, layers=2, experts=16, moe_mlp=32, q_heads=4, kv_heads=2, head_dim=16, vocab=128, E=2) -> Checkpoint:
    """Mixture-of-experts-shaped state dict (the paper's loader experiments use Qwen3 MoE
    checkpoints): per layer attention projections plus `experts` x [gate, up, down] matrices
    stored one tensor per expert, which an engine wants stacked into [experts, ...] buffers."""
    items = [("embed_tokens", (vocab, hidden), 0)]
    for l in range(layers):
        p = f"layers.{l}."
        items += [(p + "input_layernorm", (hidden,), -1), (p + "q_proj", (q_heads * head_dim, hidden), 0),
                  (p + "k_proj", (kv_heads * head_dim, hidden), 0), (p + "v_proj", (kv_heads * head_dim, hidden), 0),
                  (p + "o_proj", (hidden, q_heads * head_dim), 1), (p + "router", (experts, hidden), -1)]
        for e in range(experts):
            q = p + f"experts.{e}."
            items += [(q + "gate_proj", (moe_mlp, hidden), 0), (q + "up_proj", (moe_mlp, hidden), 0), (q + "down_proj", (hidden, moe_mlp), 1)]
    items += [("norm", (hidden,), -1), ("lm_head", (vocab, hidden), 0)]
    N = len(items)
    shapes = np.ones((N, 4), dtype=np.int64)
    ndim = np.zeros(N, dtype=np.int32)
    byte_off = np.zeros(N, dtype=np.int64)
    off = 0
    for i, (_, shp, _) in enumerate(items):
        shapes[i, :len(shp)] = shp
        ndim[i] = len(shp)
        byte_off[i] = off
        off += int(np.prod(shp)) * E
    return Checkpoint(names=[it[0] for it in items], shapes=shapes, ndim=ndim, E=np.full(N, E, dtype=np.int64),
                      byte_off=byte_off, split_dim=np.array([it[2] for it in items], dtype=np.int32), nbytes_total=off)
