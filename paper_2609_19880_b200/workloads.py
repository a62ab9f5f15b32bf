"""Seeded synthetic workloads (inputs only -- none of the method's arithmetic lives here).

Both the CPU oracle's tests and the CUDA path draw their inputs from this module so
that they see the same bits.  The tensors stand in for the captured Qwen3-8B /
Llama-3.1-8B KV caches the paper evaluates on (Sec. 5.1), which are not available:
shapes, value distributions and the paged / ragged structure follow the five
benchmark configurations, everything is drawn from a seeded ``torch.Generator``.

Conventions
  * K, V: bf16 ``[T_total, Hkv, 128]``, tokens of sequence 0 first, then 1, ...
  * q: bf16 ``[B, Hq, 128]``
  * ``seq_id[t]``, ``pos[t]``: logical sequence and position of flattened token t
  * ``slot[t] = page * 16 + offset``: physical cache slot; ``page_table[b, i]`` is
    the physical page holding tokens ``16 i .. 16 i + 15`` of sequence b
  * "N(0,3)" is a normal with standard deviation 3
"""
from __future__ import annotations

import dataclasses
import math

import torch

HEAD_DIM = 128
PAGE = 16
WINDOW = 128

# Storage budget (bits per element, averaged over K and V, one amortised INT8 mean
# byte per token-head included) -> (K record bytes, V record bytes, K levels, V levels).
# Total bytes per token-head pair = floor(32 b); keys get the paper's 2.68 : 1.84 share.
BUDGETS = {
    1.5: (27, 20, 3, 3),
    2.0: (37, 26, 4, 3),
    2.26: (42, 29, 5, 3),
    3.0: (56, 39, 8, 5),
    4.0: (75, 52, 16, 9),
}


def record_split(bits_per_elem: float):
    """(K record bytes, V record bytes) for an average budget, before any level choice."""
    total = int(math.floor(32.0 * bits_per_elem + 1e-9))
    k_rec = int(round(total * 2.68 / 4.52)) - 1
    return k_rec, total - 1 - k_rec


@dataclasses.dataclass
class Config:
    name: str
    batch: int
    hq: int
    hkv: int
    seq_lens: list
    seed: int
    k_rec: int
    v_rec: int
    k_levels: int
    v_levels: int
    alpha: float = 1.4          # < 0: automatic
    shuffle_pages: bool = False
    v_student_t: bool = False
    outliers: bool = True
    decode_steps: int = 0       # config 5: tokens appended one at a time after the prefill

    @property
    def bits_k(self):
        return self.k_rec * 8.0 / HEAD_DIM

    @property
    def bits_v(self):
        return self.v_rec * 8.0 / HEAD_DIM

    @property
    def total_tokens(self):
        return int(sum(self.seq_lens))


def make_config(idx: int, budget: float = 2.26, scale: float = 1.0) -> Config:
    """The five benchmark configurations; ``scale`` < 1 shrinks context lengths (and the
    batch of configuration 4) for quick tests while keeping structure and distributions."""
    kr, vr, km, vm = BUDGETS[budget]

    def ctx(n):
        return max(PAGE, int(n * scale))

    if idx == 1:
        return Config("c1_tiny_single_head", 1, 1, 1, [ctx(512)], 0, 36, 36, 16, 16, alpha=-1.0,
                      outliers=False)
    if idx == 2:
        return Config("c2_llama3_8b_b8_ctx8192", 8, 32, 8, [ctx(8192)] * 8, 1, kr, vr, km, vm)
    if idx == 3:
        return Config(f"c3_llama70b_ctx131072_b{budget}", 1, 64, 8, [ctx(131072)], 2, kr, vr, km, vm)
    if idx == 4:
        g = torch.Generator().manual_seed(3)
        nb = max(2, int(128 * min(1.0, scale * 4))) if scale < 1.0 else 128
        lens = torch.randint(ctx(512), ctx(16384) + 1, (nb,), generator=g).tolist()
        return Config("c4_ragged_b128_paged", nb, 32, 8, lens, 3, kr, vr, km, vm, shuffle_pages=True)
    if idx == 5:
        return Config("c5_encode_decode_loop", 4, 28, 4, [ctx(32768)] * 4, 4, kr, vr, km, vm,
                      v_student_t=True, decode_steps=max(2, int(256 * scale)) if scale < 1 else 256)
    raise ValueError(idx)


@dataclasses.dataclass
class Workload:
    cfg: Config
    k: torch.Tensor            # bf16 [T, Hkv, 128]
    v: torch.Tensor            # bf16 [T, Hkv, 128]
    q: torch.Tensor            # bf16 [B, Hq, 128]
    seq_id: torch.Tensor       # int32 [T]
    pos: torch.Tensor          # int32 [T]
    slot: torch.Tensor         # int32 [T]
    page_table: torch.Tensor   # int32 [B, max_pages]
    seq_lens: torch.Tensor     # int32 [B]
    num_pages: int
    max_windows: int
    k_offsets: torch.Tensor    # f32 [Hkv, 128] (kept for appended tokens)
    k_gain: torch.Tensor       # f32 [Hkv, 128]


def _student_t(shape, df, gen, device):
    # t = Z / sqrt(chi2_df / df), rescaled to unit variance (df > 2)
    z = torch.randn(shape, generator=gen, device=device)
    chi = torch.zeros(shape, device=device)
    for _ in range(df):
        chi += torch.randn(shape, generator=gen, device=device) ** 2
    return z / torch.sqrt(chi / df) / math.sqrt(df / (df - 2.0))


def make_kv(cfg: Config, n_tokens: int, gen, device, k_offsets, k_gain):
    """Draw K and V for n_tokens tokens (bf16), with the configuration's distributions."""
    k = torch.randn((n_tokens, cfg.hkv, HEAD_DIM), generator=gen, device=device)
    k = (k + k_offsets) * k_gain
    if cfg.v_student_t:
        v = _student_t((n_tokens, cfg.hkv, HEAD_DIM), 5, gen, device)
    else:
        v = torch.randn((n_tokens, cfg.hkv, HEAD_DIM), generator=gen, device=device)
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def generate(cfg: Config, device="cpu", extra_tokens_per_seq: int = 0) -> Workload:
    """Draw one workload.  ``extra_tokens_per_seq`` reserves page-table room (and mean
    windows) for tokens appended later (configuration 5)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev).manual_seed(cfg.seed)
    k_offsets = 3.0 * torch.randn((cfg.hkv, HEAD_DIM), generator=gen, device=dev)
    k_gain = torch.ones((cfg.hkv, HEAD_DIM), device=dev)
    if cfg.outliers:
        n_out = max(1, round(0.01 * cfg.hkv * HEAD_DIM))
        idx = torch.randperm(cfg.hkv * HEAD_DIM, generator=gen, device=dev)[:n_out]
        k_gain.view(-1)[idx] = 10.0
    T = cfg.total_tokens
    k, v = make_kv(cfg, T, gen, dev, k_offsets, k_gain)
    q = torch.randn((cfg.batch, cfg.hq, HEAD_DIM), generator=gen, device=dev).to(torch.bfloat16)

    lens = torch.tensor(cfg.seq_lens, dtype=torch.int64)
    cap = lens + extra_tokens_per_seq
    pages_per_seq = (cap + PAGE - 1) // PAGE
    max_pages = int(pages_per_seq.max())
    num_pages = int(pages_per_seq.sum())
    if cfg.shuffle_pages:
        perm = torch.randperm(num_pages, generator=torch.Generator().manual_seed(cfg.seed + 1000))
    else:
        perm = torch.arange(num_pages)
    page_table = torch.zeros((cfg.batch, max_pages), dtype=torch.int32)
    start = 0
    for b in range(cfg.batch):
        npg = int(pages_per_seq[b])
        page_table[b, :npg] = perm[start:start + npg].to(torch.int32)
        start += npg
    seq_id = torch.repeat_interleave(torch.arange(cfg.batch), lens).to(torch.int32)
    starts = torch.cumsum(lens, 0) - lens
    pos = (torch.arange(T) - torch.repeat_interleave(starts, lens)).to(torch.int32)
    slot = (page_table[seq_id.long(), (pos // PAGE).long()] * PAGE + pos % PAGE).to(torch.int32)
    max_windows = int((cap.max() + WINDOW - 1) // WINDOW)
    return Workload(cfg, k, v, q, seq_id.to(dev), pos.to(dev), slot.to(dev), page_table.to(dev),
                    lens.to(torch.int32).to(dev), num_pages, max_windows, k_offsets, k_gain)


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (host)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view("uint16")
