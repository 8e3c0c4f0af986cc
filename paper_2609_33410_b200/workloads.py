"""Seeded synthetic decode workloads (inputs only: no attention arithmetic lives here).

The paper measures on query/key/value tensors captured from real models, which cannot
be shipped; these generators stand in for them.  Shapes follow the paper's grids
(D in {64, 128}, GQA groups 1..8, 1K-128K keys, up to 256 KV heads per batch).

Recipe (every tensor drawn in FP32 from a seeded torch generator on the chosen device,
then rounded to BF16):
  q ~ N(0,1);  K, V ~ N(0,1);
  key 0 of every (request, kv head) is multiplied by `sink_gain` (an attention sink);
  a fraction `peak_frac` of the tokens j >= 1, drawn uniformly without replacement per
  (request, kv head), gets  k_j += peak_gain * q_hat,  q_hat = q / |q| of ONE query head
  of the group, chosen uniformly per boosted token.
The paged layout scatters the same logical rows into a page pool through a random
permutation of the pool's pages.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence, Union

import torch


@dataclass
class DecodeWorkload:
    q: torch.Tensor                 # [B, Hq, D] bf16
    k: torch.Tensor                 # contiguous: [B_kv, cap, Hkv, D]; paged: [pages, page_size, Hkv, D]
    v: torch.Tensor
    seqlens: torch.Tensor           # [B_kv] int32
    max_seqlen: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    stack: int = 1                  # consecutive requests sharing one KV sequence
    page_table: Optional[torch.Tensor] = None   # [B_kv, max_pages] int32, paged only
    page_size: int = 0
    scale: float = 0.0
    meta: dict = field(default_factory=dict)

    @property
    def paged(self) -> bool:
        return self.page_table is not None

    @property
    def batch(self) -> int:
        return self.q.shape[0]

    @property
    def num_seqs(self) -> int:
        return self.seqlens.shape[0]

    def cache_bytes(self) -> int:
        """Full-cache bytes: sum_b n_b * Hkv * 4D (BF16 key + value rows)."""
        return int(self.seqlens.to(torch.int64).sum().item()) * self.num_kv_heads * 4 * self.head_dim

    def logical_rows(self, which: str, seq: int, kvh: int) -> torch.Tensor:
        """Logical [n, D] bf16 rows of one (KV sequence, kv head), hiding the layout."""
        t = self.k if which == "k" else self.v
        n = int(self.seqlens[seq].item())
        if not self.paged:
            return t[seq, :n, kvh]
        j = torch.arange(n, device=t.device)
        pages = self.page_table[seq].to(torch.int64)[j // self.page_size]
        return t[pages, j % self.page_size, kvh]


def bf16_bits(t: torch.Tensor):
    """numpy uint16 view of a bf16 tensor's bit patterns (for exact widening on the CPU)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")


def make_decode_workload(batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int,
                         seqlens: Union[int, Sequence[int]], seed: int = 0,
                         device: Union[str, torch.device] = "cpu", paged: bool = False,
                         page_size: int = 64, sink_gain: float = 8.0, peak_frac: float = 0.01,
                         peak_gain: float = 4.0, stack: int = 1, capacity: Optional[int] = None,
                         poison_padding: bool = False, q: Optional[torch.Tensor] = None) -> DecodeWorkload:
    """Build one workload.  `batch` counts requests; there are batch // stack KV sequences
    (stack > 1: `stack` consecutive requests read the same KV sequence, as the shared
    prefix level of a cascade does).  `seqlens` is an int or one length per KV sequence.
    `poison_padding` fills rows beyond each length (and unused page tails) with NaN so a
    test can prove they are masked.  `q` lets two levels of a cascade share queries."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    B, Hq, Hkv, D = batch, num_q_heads, num_kv_heads, head_dim
    assert Hq % Hkv == 0 and B % stack == 0
    G = Hq // Hkv
    Bkv = B // stack
    lens = [int(seqlens)] * Bkv if isinstance(seqlens, int) else [int(x) for x in seqlens]
    assert len(lens) == Bkv
    max_len = max(lens) if lens else 0
    if q is None:
        q = torch.randn(B, Hq, D, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    qf = q.to(torch.float32)
    qhat = qf / qf.norm(dim=-1, keepdim=True).clamp_min(1e-20)          # [B, Hq, D]

    if paged:
        pages_per_seq = [(n + page_size - 1) // page_size for n in lens]
        max_pages = max(pages_per_seq) if pages_per_seq else 0
        total_pages = sum(pages_per_seq)
        perm = torch.randperm(max(total_pages, 1), generator=g, device=dev)
        table = torch.zeros(Bkv, max(max_pages, 1), dtype=torch.int32, device=dev)
        fill = float("nan") if poison_padding else 0.0
        kpool = torch.full((max(total_pages, 1), page_size, Hkv, D), fill, dtype=torch.bfloat16, device=dev)
        vpool = torch.full_like(kpool, fill)
        cap = 0
    else:
        cap = int(capacity) if capacity is not None else max_len
        assert cap >= max_len
        fill = float("nan") if poison_padding else 0.0
        kc = torch.full((Bkv, max(cap, 1), Hkv, D), fill, dtype=torch.bfloat16, device=dev)
        vc = torch.full_like(kc, fill)

    page_cursor = 0
    for s, n in enumerate(lens):
        if n == 0:
            continue
        kf = torch.randn(n, Hkv, D, generator=g, device=dev, dtype=torch.float32)
        vf = torch.randn(n, Hkv, D, generator=g, device=dev, dtype=torch.float32)
        kf[0] *= sink_gain
        n_peak = int(round(peak_frac * (n - 1))) if n > 1 else 0
        if n_peak > 0:
            for h in range(Hkv):
                tok = torch.randperm(n - 1, generator=g, device=dev)[:n_peak] + 1
                # one query row of the group (and of the stacked requests) per boosted token
                pick_r = torch.randint(0, stack, (n_peak,), generator=g, device=dev) + s * stack
                pick_h = torch.randint(0, G, (n_peak,), generator=g, device=dev) + h * G
                kf[tok, h] += peak_gain * qhat[pick_r, pick_h]
        kb, vb = kf.to(torch.bfloat16), vf.to(torch.bfloat16)
        if paged:
            npg = pages_per_seq[s]
            ids = perm[page_cursor:page_cursor + npg]
            page_cursor += npg
            table[s, :npg] = ids.to(torch.int32)
            pad = npg * page_size - n
            if pad:
                padrow = torch.full((pad, Hkv, D), fill, dtype=torch.bfloat16, device=dev)
                kb = torch.cat([kb, padrow]); vb = torch.cat([vb, padrow])
            kpool[ids] = kb.view(npg, page_size, Hkv, D)
            vpool[ids] = vb.view(npg, page_size, Hkv, D)
        else:
            kc[s, :n] = kb
            vc[s, :n] = vb
        del kf, vf, kb, vb

    seqlens_t = torch.tensor(lens, dtype=torch.int32, device=dev)
    meta = dict(seed=seed, sink_gain=sink_gain, peak_frac=peak_frac, peak_gain=peak_gain)
    if paged:
        return DecodeWorkload(q, kpool, vpool, seqlens_t, max_len, Hq, Hkv, D, stack, table, page_size,
                              1.0 / D ** 0.5, meta)
    return DecodeWorkload(q, kc, vc, seqlens_t, max_len, Hq, Hkv, D, stack, None, 0, 1.0 / D ** 0.5, meta)


def make_cascade_workload(batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, prefix_len: int,
                          suffix_lens: Union[int, Sequence[int]], seed: int = 0, device="cpu", **kw):
    """Requests that share one prefix and own private suffixes.  Returns (prefix level, suffix level):
    two workloads over the same queries; the prefix level stacks all requests on one KV sequence."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    q = torch.randn(batch, num_q_heads, head_dim, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    pre = make_decode_workload(batch, num_q_heads, num_kv_heads, head_dim, prefix_len, seed=seed + 1, device=dev,
                               stack=batch, q=q, **kw)
    suf = make_decode_workload(batch, num_q_heads, num_kv_heads, head_dim, suffix_lens, seed=seed + 2, device=dev,
                               q=q, sink_gain=1.0, **kw)
    return pre, suf


def make_draft_workload(num_seqs: int, draft_len: int, num_q_heads: int, num_kv_heads: int, head_dim: int,
                        context_lens: Union[int, Sequence[int]], seed: int = 0, device="cpu", tree: bool = False, **kw):
    """Draft / tree verification: every sequence holds its committed context followed by `draft_len` draft tokens,
    and `draft_len` requests (stacked on the sequence) verify them.  Returns (workload, masks, draft_len): request
    seq * draft_len + r is draft row r; bit t of masks[request] says whether it uses draft key t.
    Chain: row r uses drafts 0..r.  Tree: a random parent among the earlier drafts (or none) per draft; a row uses
    its ancestors and itself.  Masks are int32 bit patterns."""
    m = int(draft_len)
    assert 1 <= m <= 32
    ctx = [int(context_lens)] * num_seqs if isinstance(context_lens, int) else [int(x) for x in context_lens]
    w = make_decode_workload(num_seqs * m, num_q_heads, num_kv_heads, head_dim, [c + m for c in ctx], seed=seed,
                             device=device, stack=m, **kw)
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) + 977)
    masks = []
    for _ in range(num_seqs):
        row = []
        for r in range(m):
            if tree:
                parent = int(torch.randint(-1, r, (1,), generator=g).item()) if r > 0 else -1
                anc = row[parent] if parent >= 0 else 0
            else:
                anc = row[r - 1] if r > 0 else 0
            row.append(anc | (1 << r))
        masks += row
    t = torch.tensor([x - (1 << 32) if x >= (1 << 31) else x for x in masks], dtype=torch.int32, device=device)
    return w, t, m


# The five benchmark configurations, by name.  `scale_down` shrinks context (and for the
# sweep the batch) so the CPU oracle can check every row in seconds.
def config_workload(name: str, device="cpu", small: bool = False, **over) -> DecodeWorkload:
    if name == "c1":      # MHA, batch 1, 8 heads, D=128, 4096 keys, sink only
        kw = dict(batch=1, num_q_heads=8, num_kv_heads=8, head_dim=128, seqlens=4096, seed=0, peak_frac=0.0)
    elif name == "c2":    # GQA 32/8, batch 16, 32768 keys, peaked keys
        kw = dict(batch=16, num_q_heads=32, num_kv_heads=8, head_dim=128, seqlens=32768, seed=1)
        if small:
            kw.update(batch=2, seqlens=4096 + 37)
    elif name == "c3":    # GQA 32/8, batch 4, 131072 keys, paged (64-token pages, random permutation)
        kw = dict(batch=4, num_q_heads=32, num_kv_heads=8, head_dim=128, seqlens=131072, seed=2,
                  paged=True, page_size=64)
        if small:
            kw.update(batch=2, seqlens=8192 + 100)
    else:
        raise KeyError(name)
    kw.update(over)
    return make_decode_workload(device=device, **kw)
