"""Seeded synthetic inputs for the PPSA decode-attention path.

This module only draws numbers and lays them out in memory; it contains none of
the method's arithmetic (no attention, no top-k) and is the one piece of code
that both the CUDA tests/benchmark and the CPU oracle's tests may share. Values
are generated once, on the device asked for, and the bits are copied wherever
else they are needed; nothing is ever regenerated on a second device.

The shapes stand in for the Llama-2-7B / Llama-3-8B decode workloads the paper
evaluates (Section 4): bf16 N(0,1) queries, keys and values, plus a few
"heavy hitter" positions per KV head whose keys are correlated with the query
(key = 0.5 * q_hat + noise, q_hat = q rescaled to unit RMS) so that the top of
the score distribution is well separated, as it is in a trained model.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

LAYER_FULL, LAYER_SELECT, LAYER_SPARSE = 0, 1, 2
BASE_SEED = 241005076
PAGE_SIZE = 16


def schedule(num_layers: int, reselect_layer: int = 13) -> List[int]:
    """Layer types of one decode step: two full layers, a selection layer at
    layer 2 and at `reselect_layer` (0-based), sparse layers elsewhere
    (Section 3, Figure 2; Section 4.3 for the 2+2+28 / 2+2+60 mix)."""
    out = []
    for i in range(num_layers):
        if i < 2:
            out.append(LAYER_FULL)
        elif i == 2 or i == reselect_layer:
            out.append(LAYER_SELECT)
        else:
            out.append(LAYER_SPARSE)
    return out


@dataclass
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    num_layers: int
    ctx: int                      # context length (max over the batch when ragged)
    k: int                        # token budget
    planted: int                  # heavy-hitter positions per (layer, KV head)
    sched: List[int]
    seed: int
    head_dim: int = 128
    paged: bool = False
    ragged: bool = False          # per-sequence lengths drawn from [ctx_min, ctx]
    ctx_min: int = 0

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    def ctx_lens(self) -> List[int]:
        if not self.ragged:
            return [self.ctx] * self.batch
        g = torch.Generator(device="cpu").manual_seed(self.seed + 7)
        span = self.ctx - self.ctx_min + 1
        return [int(self.ctx_min + int(x)) for x in torch.randint(0, span, (self.batch,), generator=g)]


def workload(name: str) -> Workload:
    """The five benchmark configurations, plus 'tiny' variants used by tests."""
    if name == "cfg1":    # one selection layer followed by one sparse layer, GQA group 4
        return Workload(name, 1, 8, 2, 2, 4096, 256, 32, [LAYER_SELECT, LAYER_SPARSE], BASE_SEED + 1)
    if name == "cfg2":    # Llama-2-7B attention shapes (MHA)
        return Workload(name, 1, 32, 32, 32, 32768, 2048, 64, schedule(32, 13), BASE_SEED + 2)
    if name == "cfg3":    # Llama-3-8B attention shapes (GQA 32/8), 128K context
        return Workload(name, 1, 32, 8, 32, 131072, 4096, 64, schedule(32, 13), BASE_SEED + 3)
    if name == "cfg4":    # batched paged decode, ragged lengths
        return Workload(name, 8, 32, 8, 32, 65536, 2048, 64, schedule(32, 13), BASE_SEED + 4,
                        paged=True, ragged=True, ctx_min=8192)
    if name == "cfg64":   # the 64-layer variant of Section 4.3 (2 + 2 + 60): Llama-3-70B attention shapes, GQA group 8,
        #                   32K context (the longest the paper runs that model at), re-selection at layer 31
        return Workload(name, 1, 64, 8, 64, 32768, 2048, 64, schedule(64, 31), BASE_SEED + 6)
    raise KeyError(name)


def sweep_point(ctx: int, k: int) -> Workload:
    """One point of the context x budget sweep: Llama-3-8B head shapes, one
    selection layer followed by one sparse layer."""
    return Workload(f"cfg5_n{ctx}_k{k}", 1, 32, 8, 2, ctx, k, 64, [LAYER_SELECT, LAYER_SPARSE],
                    BASE_SEED + 5)


SWEEP_CTX = (4096, 16384, 65536, 131072, 262144)
SWEEP_K = (512, 1024, 2048, 4096, 8192)


@dataclass
class LayerKV:
    """One layer's KV cache and its addressing (all strides in elements).

    contiguous: element (b, pos, g, c) of K at k.data_ptr + 2*(b*stride_b +
    pos*stride_pos + g*stride_head + c); paged: page = page_table[b, pos // 16],
    slot = pos % 16, element at page*stride_page + slot*stride_pos +
    g*stride_head + c. V uses the same strides from its own base."""
    k: torch.Tensor               # base tensors; k and v may be views of one buffer
    v: torch.Tensor
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    ctx_lens: torch.Tensor        # int32 [B] on the same device
    max_ctx_len: int
    stride_b: int = 0
    stride_pos: int = 0
    stride_head: int = 0
    stride_page: int = 0
    page_table: Optional[torch.Tensor] = None   # int32 [B, max_pages_per_seq]
    page_size: int = PAGE_SIZE
    max_pages_per_seq: int = 0
    sm_scale: float = 0.0
    keep: list = field(default_factory=list)    # owning buffers
    kv_dtype: int = 0                           # 0: bf16; 1: OCP FP8 E4M3 codes with per-KV-head scales
    k_scale: Optional[torch.Tensor] = None      # float32 [Hkv] on the device (fp8 only)
    v_scale: Optional[torch.Tensor] = None

    @property
    def paged(self) -> bool:
        return self.page_table is not None

    def kv_bytes(self) -> int:
        """Bytes of K and V that a full pass over the cache must read."""
        return int(self.ctx_lens.sum().item()) * self.num_kv_heads * self.head_dim * 2 * (1 if self.kv_dtype else 2)


def _gen(device, seed: int) -> torch.Generator:
    return torch.Generator(device=device).manual_seed(seed)


def make_q(w: Workload, layer: int, device) -> torch.Tensor:
    g = _gen(device, w.seed * 1000 + layer * 10 + 1)
    return torch.randn(w.batch, w.num_q_heads, w.head_dim, generator=g, device=device,
                       dtype=torch.float32).to(torch.bfloat16)


def planted_positions(w: Workload, layer: int, ctx_lens: Sequence[int]) -> torch.Tensor:
    """int64 [B, Hkv, P] distinct positions per (sequence, KV head): the first
    half is the same for every layer (tokens that stay important across
    layers), the second half is redrawn per layer. Always drawn on the CPU so
    that they do not depend on the device."""
    P = w.planted
    out = torch.zeros(w.batch, w.num_kv_heads, P, dtype=torch.int64)
    for b in range(w.batch):
        n = ctx_lens[b]
        p = min(P, n)
        for g in range(w.num_kv_heads):
            shared = torch.randperm(n, generator=_gen("cpu", w.seed * 77 + b * 131 + g))[:p]
            own = torch.randperm(n, generator=_gen("cpu", w.seed * 77 + b * 131 + g + 100003 * (layer + 1)))
            half = p // 2
            taken = set(shared[:half].tolist())
            rest = [x for x in own[: 2 * p].tolist() if x not in taken][: p - half]
            pos = shared[:half].tolist() + rest
            out[b, g, :p] = torch.tensor(pos, dtype=torch.int64)
            if p < P:
                out[b, g, p:] = out[b, g, 0]
    return out


def _plant(w: Workload, q: torch.Tensor, kview_of, layer: int, ctx_lens: Sequence[int]) -> None:
    """Overwrite the K rows at the planted positions with 0.5*q_hat + (row)."""
    pos = planted_positions(w, layer, ctx_lens)
    G = w.group
    qf = q.float()
    qhat = qf * (w.head_dim ** 0.5) / qf.norm(dim=-1, keepdim=True).clamp_min(1e-20)
    for b in range(w.batch):
        for g in range(w.num_kv_heads):
            rows = kview_of(b, g)                       # [N_b, d] view into the cache
            p = pos[b, g].to(rows.device)
            heads = g * G + (torch.arange(w.planted) % G)
            target = qhat[b, heads.to(q.device)]        # [P, d]
            rows[p] = (0.5 * target + rows[p].float()).to(torch.bfloat16)


def make_layer(w: Workload, layer: int, device, layout: str = "hnd_interleaved",
               q: Optional[torch.Tensor] = None, page_table: Optional[torch.Tensor] = None,
               num_pages: int = 0) -> LayerKV:
    """Build one layer's cache with planted heavy hitters.

    layout: 'hnd_interleaved'  [B][Hkv][N][2(K|V)][d]  (one position = 512 contiguous bytes)
            'nhd_separate'     K and V each [B][N][Hkv][d]
            'paged'            pool [page][Hkv][16][2][d] + page table"""
    d, B, Hkv = w.head_dim, w.batch, w.num_kv_heads
    lens = w.ctx_lens()
    N = w.ctx
    if q is None:
        q = make_q(w, layer, device)
    g = _gen(device, w.seed * 1000 + layer * 10 + 2)
    ctx_t = torch.tensor(lens, dtype=torch.int32, device=device)
    common = dict(batch=B, num_q_heads=w.num_q_heads, num_kv_heads=Hkv, head_dim=d,
                  ctx_lens=ctx_t, max_ctx_len=N)
    if layout == "hnd_interleaved":
        buf = torch.empty(B, Hkv, N, 2, d, dtype=torch.bfloat16, device=device)
        buf.normal_(generator=g)
        _plant(w, q, lambda b, h: buf[b, h, : lens[b], 0, :], layer, lens)
        return LayerKV(k=buf[:, :, :, 0, :], v=buf[:, :, :, 1, :], stride_b=Hkv * N * 2 * d,
                       stride_pos=2 * d, stride_head=N * 2 * d, keep=[buf], **common)
    if layout == "nhd_separate":
        kb = torch.empty(B, N, Hkv, d, dtype=torch.bfloat16, device=device)
        vb = torch.empty(B, N, Hkv, d, dtype=torch.bfloat16, device=device)
        kb.normal_(generator=g)
        vb.normal_(generator=g)
        _plant(w, q, lambda b, h: kb[b, : lens[b], h, :], layer, lens)
        return LayerKV(k=kb, v=vb, stride_b=N * Hkv * d, stride_pos=Hkv * d, stride_head=d,
                       keep=[kb, vb], **common)
    if layout == "paged":
        assert page_table is not None
        pool = torch.empty(num_pages, Hkv, PAGE_SIZE, 2, d, dtype=torch.bfloat16, device=device)
        pool.normal_(generator=g)
        pt = page_table.to(device)
        pos = planted_positions(w, layer, lens)
        G = w.group
        qf = q.float()
        qhat = qf * (d ** 0.5) / qf.norm(dim=-1, keepdim=True).clamp_min(1e-20)
        for b in range(B):
            for h in range(Hkv):
                p = pos[b, h].to(device)
                pages = pt[b, (p // PAGE_SIZE)].long()
                slots = p % PAGE_SIZE
                heads = (h * G + (torch.arange(w.planted) % G)).to(device)
                rows = pool[pages, h, slots, 0, :].float()
                pool[pages, h, slots, 0, :] = (0.5 * qhat[b, heads] + rows).to(torch.bfloat16)
        return LayerKV(k=pool[:, :, :, 0, :], v=pool[:, :, :, 1, :], stride_pos=2 * d,
                       stride_head=PAGE_SIZE * 2 * d, stride_page=Hkv * PAGE_SIZE * 2 * d,
                       page_table=pt.to(torch.int32).contiguous(), max_pages_per_seq=pt.shape[1],
                       keep=[pool], **common)
    raise ValueError(layout)


KV_BF16, KV_FP8_E4M3 = 0, 1


def to_fp8(layer: LayerKV, k_scale: Optional[torch.Tensor] = None, v_scale: Optional[torch.Tensor] = None) -> LayerKV:
    """The same cache stored as OCP FP8 E4M3 codes (torch's float8_e4m3fn cast: round to nearest even,
    saturating) with one scale per KV head for K and one for V: code = cast(value / scale). The default
    scales map each KV head's largest magnitude to 240, a little over half of the format's range. The
    buffer keeps its layout; element strides stay what they were, rows are half as long in bytes.
    Data preparation only (a storage format), no arithmetic of the method."""
    assert layer.kv_dtype == KV_BF16 and len(layer.keep) == 1, "needs a cache held in one buffer"
    buf = layer.keep[0]
    Hkv, dev = layer.num_kv_heads, buf.device
    paged = layer.page_table is not None
    hdim = 1                                       # [B][Hkv][N][2][d] and [page][Hkv][16][2][d]: heads are dim 1
    kview, vview = buf.select(-2, 0), buf.select(-2, 1)
    red = [i for i in range(kview.dim()) if i != hdim]
    if k_scale is None:
        k_scale = (kview.float().abs().amax(dim=red) / 240.0).clamp_min(2.0 ** -20)
    if v_scale is None:
        v_scale = (vview.float().abs().amax(dim=red) / 240.0).clamp_min(2.0 ** -20)
    k_scale, v_scale = k_scale.to(dev, torch.float32), v_scale.to(dev, torch.float32)
    shape = [1] * buf.dim()
    shape[hdim] = Hkv
    q8 = torch.empty(buf.shape, dtype=torch.float8_e4m3fn, device=dev)
    q8.select(-2, 0).copy_((kview.float() / k_scale.view(shape[:-1])).to(torch.float8_e4m3fn))
    q8.select(-2, 1).copy_((vview.float() / v_scale.view(shape[:-1])).to(torch.float8_e4m3fn))
    out = LayerKV(k=q8.select(-2, 0), v=q8.select(-2, 1), batch=layer.batch, num_q_heads=layer.num_q_heads,
                  num_kv_heads=Hkv, head_dim=layer.head_dim, ctx_lens=layer.ctx_lens, max_ctx_len=layer.max_ctx_len,
                  stride_b=layer.stride_b, stride_pos=layer.stride_pos, stride_head=layer.stride_head,
                  stride_page=layer.stride_page, page_table=layer.page_table, page_size=layer.page_size,
                  max_pages_per_seq=layer.max_pages_per_seq, sm_scale=layer.sm_scale, keep=[q8],
                  kv_dtype=KV_FP8_E4M3, k_scale=k_scale, v_scale=v_scale)
    if paged:
        out.num_pages = getattr(layer, "num_pages", 0) or buf.shape[0]
    return out


def make_page_table(w: Workload, extra_pages: int = 0):
    """One page table shared by all layers: each sequence's logical pages are a
    slice of one seeded shuffle of all physical pages. Returns (int32 [B, max_pages]
    CPU tensor padded with page 0, number of physical pages)."""
    lens = w.ctx_lens()
    need = [(n + PAGE_SIZE - 1) // PAGE_SIZE for n in lens]
    total = sum(need) + extra_pages
    perm = torch.randperm(total, generator=_gen("cpu", w.seed + 99))
    maxp = (w.ctx + PAGE_SIZE - 1) // PAGE_SIZE      # table width covers the declared maximum length
    pt = torch.zeros(w.batch, maxp, dtype=torch.int32)
    at = 0
    for b, nb in enumerate(need):
        pt[b, :nb] = perm[at: at + nb].to(torch.int32)
        at += nb
    return pt, total


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array holding the same bits; fp8 tensor -> uint8 codes (host copy)."""
    if t.element_size() == 1:
        return t.detach().contiguous().view(torch.uint8).cpu().numpy()
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view("uint16")
