"""Seeded synthetic inputs for the OasisKV decode hot path.

This module only draws random numbers and lays them out; it contains none of the
method's arithmetic (no summaries, scores, selection or attention), so both the CUDA
library and the CPU checker can be fed from it.

Shapes follow the paper's Qwen3-8B-like evaluation setting (Sec. 5.2: 16-token blocks,
K = 128 selected blocks plus the active local block; 32 query / 8 KV heads of
dimension 128) and the five benchmark configurations built on it.  The paper's
datasets and model weights are not used: planted "heavy-hitter" blocks stand in for
the skewed attention of real traces (Sec. 2.2) and "true query + noise" stands in for
the speculative draft queries (Sec. 4.2.1).

Layouts
  host_kv      [n_phys_blocks][Hkv][2][16][128] bf16   (2 = K part, V part)
  block_table  [B][max_blocks] int32  logical -> physical block
  q            [B][T][Hq][128] bf16   token 0 = verified token, 1..Td = draft tokens
  q_true       [B][Td][Hq][128] bf16  the true next-step queries the drafts approximate
"""
from dataclasses import dataclass, field, replace
from typing import Optional

import torch

HEAD_DIM = 128
BLOCK = 16


@dataclass(frozen=True)
class Config:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    context: int              # history tokens L at the first step (multiple of 16)
    k_blocks: int             # K = budget tokens / 16
    n_draft: int              # Td
    layers: int = 1
    steps: int = 1            # consecutive decode steps (drift workload only)
    density: float = 0.05     # share of blocks that are planted heavy hitters
    plant_scale: float = 3.0
    noise: float = 0.1        # std of the draft-query noise
    zipf: float = 0.0         # > 0: r-th heavy block scaled by r**-zipf
    drift: int = 0            # > 0: hot set moves by up to +-drift blocks per step
    ar_rho: float = 0.9       # AR(1) coefficient of the query background (drift only)
    config_id: int = 0
    head_dim: int = HEAD_DIM
    block_size: int = BLOCK

    @property
    def n_q_tokens(self):     # T
        return self.n_draft + 1

    @property
    def group(self):          # G
        return self.n_q_heads // self.n_kv_heads

    @property
    def max_blocks(self):
        # room for every token that any step of the workload can touch, rounded up to 8
        last = self.context + self.steps - 1 + self.n_q_tokens + self.n_draft
        nb = (last + self.block_size - 1) // self.block_size
        return (nb + 7) // 8 * 8


# The five benchmark configurations (full size).
C1 = Config("c1_single", 1, 32, 8, 8192, 128, 4, layers=1, density=0.05, config_id=1)
C2 = Config("c2_reasoning", 16, 32, 8, 32768, 128, 4, layers=32, steps=64, density=0.03,
            drift=64, config_id=2)
C3 = Config("c3_longctx", 32, 32, 8, 131072, 128, 4, layers=4, density=0.01, zipf=1.1,
            config_id=3)
C4 = Config("c4_gqa8", 8, 64, 8, 65536, 256, 8, layers=8, density=0.05, noise=0.2,
            config_id=4)
C5 = Config("c5_sweep", 16, 32, 8, 65536, 128, 4, layers=1, density=0.05, config_id=5)
CONFIGS = {c.name: c for c in (C1, C2, C3, C4, C5)}


def scaled(cfg: Config, **kw) -> Config:
    """A smaller (or otherwise modified) variant of a configuration."""
    return replace(cfg, **kw)


@dataclass
class Layer:
    """Inputs of one layer of one workload (first decode step unless stated)."""
    cfg: Config
    host_kv: torch.Tensor
    block_table: torch.Tensor
    seq_len: torch.Tensor          # [B] int32, history tokens L_b
    n_full: torch.Tensor           # [B] int32, full blocks floor(L_b/16)
    q: torch.Tensor                # [B][T][Hq][d]
    q_true: torch.Tensor           # [B][Td][Hq][d]
    # drift workload: per-step tensors, index 0 = the fields above
    q_steps: Optional[torch.Tensor] = None        # [S][B][T][Hq][d]
    q_true_steps: Optional[torch.Tensor] = None   # [S][B][Td][Hq][d]
    seq_len_steps: Optional[torch.Tensor] = None  # [S][B]
    n_full_steps: Optional[torch.Tensor] = None   # [S][B]
    extra: dict = field(default_factory=dict)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _unit(x):
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-12)


def layer_seed(cfg: Config, seed: int, layer: int) -> int:
    return int(seed) + 1000 * cfg.config_id + layer


def make_layer(cfg: Config, seed: int = 0, layer: int = 0, device="cpu", pin: bool = False,
               permute_table: bool = False, ragged: bool = False,
               out_kv: Optional[torch.Tensor] = None) -> Layer:
    """Draws one layer's KV pool and queries.

    The KV pool is drawn request by request on `device` and copied into one host
    tensor (pinned when `pin`), or into `out_kv` when the caller supplies the storage.
    `ragged` gives the requests different history lengths (test use); `permute_table`
    replaces the identity block table by a seeded permutation of the physical blocks.
    """
    B, Hq, Hkv, d, bs = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.block_size
    G, T, Td, mb = cfg.group, cfg.n_q_tokens, cfg.n_draft, cfg.max_blocks
    S = cfg.steps
    base = layer_seed(cfg, seed, layer)
    gc = _gen("cpu", base)              # small things are always drawn on the CPU

    # history lengths
    if ragged:
        lens = torch.randint(max(bs, cfg.context // 2), cfg.context + 1, (B,), generator=gc)
        lens[0] = cfg.context
    else:
        lens = torch.full((B,), cfg.context, dtype=torch.int64)
    seq_len_steps = (lens[None, :] + torch.arange(S)[:, None]).to(torch.int32)   # [S][B]
    n_full_steps = (seq_len_steps // bs).to(torch.int32)

    # block table
    P = B * mb
    if permute_table:
        block_table = torch.randperm(P, generator=gc).to(torch.int32).view(B, mb)
    else:
        block_table = torch.arange(P, dtype=torch.int32).view(B, mb)

    # planted structure
    u = _unit(torch.randn(B, Hkv, d, generator=gc))                  # shared direction per (b,h)
    plant = torch.zeros(B, Hkv, mb)                                   # scale of u added to keys
    block_dir = None
    hot_steps = None
    if cfg.drift > 0:
        # every block carries its own direction; the hot set only exists in the queries
        block_dir = _unit(torch.randn(B, Hkv, mb, d, generator=gc))
        n_hot = max(1, int(round(cfg.density * (cfg.context // bs))))
        hot = torch.stack([torch.stack([torch.randperm(int(lens[b]) // bs, generator=gc)[:n_hot]
                                        for _ in range(Hkv)]) for b in range(B)])   # [B][Hkv][n_hot]
        hot_steps = [hot]
        for s in range(1, S + Td + 1):
            step = torch.randint(-cfg.drift, cfg.drift + 1, hot.shape, generator=gc)
            hi = ((lens + s) // bs - 1).view(B, 1, 1)
            nxt = hot_steps[-1] + step
            nxt = torch.where(nxt < 0, -nxt, nxt)
            nxt = torch.where(nxt > hi, 2 * hi - nxt, nxt).clamp_min(0)
            hot_steps.append(nxt)
    else:
        for b in range(B):
            nf = int(lens[b]) // bs
            n_heavy = max(1, int(round(cfg.density * nf)))
            for h in range(Hkv):
                chosen = torch.randperm(nf, generator=gc)[:n_heavy]
                if cfg.zipf > 0:
                    r = torch.arange(1, n_heavy + 1, dtype=torch.float32)
                    plant[b, h, chosen] = cfg.plant_scale * r.pow(-cfg.zipf)
                else:
                    plant[b, h, chosen] = cfg.plant_scale

    # KV pool, request by request
    if out_kv is not None:
        host_kv = out_kv
        assert tuple(host_kv.shape) == (P, Hkv, 2, bs, d) and host_kv.dtype == torch.bfloat16
    else:
        host_kv = torch.empty((P, Hkv, 2, bs, d), dtype=torch.bfloat16, pin_memory=pin)
    gd = _gen(device, base + 7919)
    for b in range(B):
        kv = torch.randn((mb, Hkv, 2, bs, d), generator=gd, device=device, dtype=torch.float32)
        if block_dir is not None:
            add = cfg.plant_scale * block_dir[b].to(device).permute(1, 0, 2)          # [mb][Hkv][d]
        else:
            add = (plant[b].to(device).t()[:, :, None] * u[b].to(device)[None, :, :])  # [mb][Hkv][d]
        kv[:, :, 0] += add[:, :, None, :]
        kv = kv.to(torch.bfloat16)
        phys = block_table[b].to(torch.int64)
        if permute_table:
            host_kv[phys] = kv.cpu()
        else:
            host_kv[b * mb:(b + 1) * mb].copy_(kv)
        del kv

    # queries: true next-step queries, their noisy drafts, and the verified token's query
    def head_signal(sig_bh):      # [B][Hkv][d] -> [B][Hq][d]
        return sig_bh.repeat_interleave(G, dim=1)

    n_q_steps = S + Td + 1
    if cfg.drift > 0:
        z = torch.randn(B, Hq, d, generator=gc)
        truth = []
        rho = cfg.ar_rho
        for s in range(n_q_steps):
            idx = hot_steps[s]                                                    # [B][Hkv][n_hot]
            sig = torch.gather(block_dir, 2, idx[..., None].expand(-1, -1, -1, d)).sum(dim=2)
            truth.append(z + cfg.plant_scale * head_signal(sig))
            z = rho * z + (1.0 - rho * rho) ** 0.5 * torch.randn(B, Hq, d, generator=gc)
        truth = torch.stack(truth)                                                # [S+Td+1][B][Hq][d]
    else:
        z = torch.randn(n_q_steps, B, Hq, d, generator=gc)
        truth = z + cfg.plant_scale * head_signal(u)[None]

    q_steps = torch.empty(S, B, T, Hq, d)
    q_true_steps = torch.empty(S, B, Td, Hq, d)
    for s in range(S):
        nxt = truth[s + 1:s + 1 + Td].permute(1, 0, 2, 3)                         # [B][Td][Hq][d]
        q_true_steps[s] = nxt
        q_steps[s, :, 0] = truth[s]
        q_steps[s, :, 1:] = nxt + cfg.noise * torch.randn(B, Td, Hq, d, generator=gc)
    q_steps = q_steps.to(torch.bfloat16)
    q_true_steps = q_true_steps.to(torch.bfloat16)

    extra = {"plant": plant, "u": u}
    if hot_steps is not None:
        extra["hot_steps"] = hot_steps
    return Layer(cfg=cfg, host_kv=host_kv, block_table=block_table,
                 seq_len=seq_len_steps[0].contiguous(), n_full=n_full_steps[0].contiguous(),
                 q=q_steps[0].contiguous(), q_true=q_true_steps[0].contiguous(),
                 q_steps=q_steps, q_true_steps=q_true_steps,
                 seq_len_steps=seq_len_steps.contiguous(), n_full_steps=n_full_steps.contiguous(),
                 extra=extra)


def new_kv_steps(lay: Layer, kv: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The keys and values each step appends, read out of the pre-generated pool: element [s][b][t][h] is the
    (key row, value row) of position seq_len_steps[s][b] + t.  Shape [S][B][T][Hkv][2][d], on kv's device."""
    cfg = lay.cfg
    kv = lay.host_kv if kv is None else kv
    pos = lay.seq_len_steps.to(torch.int64)[:, :, None] + torch.arange(cfg.n_q_tokens)[None, None, :]   # [S][B][T]
    blk, row = pos // cfg.block_size, pos % cfg.block_size
    phys = torch.gather(lay.block_table.to(torch.int64)[None].expand(pos.shape[0], -1, -1), 2, blk)
    return kv[phys.to(kv.device), :, :, row.to(kv.device)].contiguous()


def blank_future(kv: torch.Tensor, lay: Layer) -> torch.Tensor:
    """Zeroes, in place, every position of the pool at or beyond each request's first-step history length: the
    state of a cache whose later tokens have not been produced yet."""
    cfg = lay.cfg
    bs = cfg.block_size
    for b in range(cfg.batch):
        L = int(lay.seq_len_steps[0][b])
        lo = L // bs
        table = lay.block_table[b].to(torch.int64)
        if L % bs:
            kv[table[lo], :, :, L % bs:] = 0
            lo += 1
        kv[table[lo:]] = 0
    return kv


def u16(t: torch.Tensor):
    """bf16 CPU tensor -> numpy uint16 bit patterns (shares memory)."""
    import numpy as np
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_u16(a) -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 CPU tensor."""
    import numpy as np
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16).copy()).view(torch.bfloat16)
