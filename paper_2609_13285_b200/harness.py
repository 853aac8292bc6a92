"""Moves a generated decode case into device memory and wraps the three library calls.

No arithmetic happens here: tensors are uploaded as generated (bf16 pools as raw 16-bit patterns, e4m3 pools as bytes)
and handed to the C ABI through `binding`.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import binding as gb
from .workloads import DecodeCase


def _dev(a: Optional[np.ndarray], device) -> Optional[torch.Tensor]:
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device)   # raw bf16 bit patterns
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


@dataclass
class DeviceCase:
    case: DecodeCase
    handle: int
    v_pool: torch.Tensor
    kr_pool: torch.Tensor
    block_table: Optional[torch.Tensor]
    seq_lens: torch.Tensor
    q_c: torch.Tensor
    q_r: torch.Tensor
    M: torch.Tensor
    q_pos: torch.Tensor
    v_new: torch.Tensor
    kr_new: torch.Tensor
    append_pos: torch.Tensor
    q_abs: torch.Tensor
    out: torch.Tensor
    lse: torch.Tensor
    status: torch.Tensor
    workspace: Optional[torch.Tensor] = None
    workspace_splits: int = -1

    @property
    def cache(self) -> gb.GvaCache:
        c = self.case
        return gb.make_cache(self.v_pool, self.kr_pool, self.block_table, c.num_pages, c.max_pages_per_seq)

    def ensure_workspace(self, num_splits: int) -> torch.Tensor:
        need = gb.gva_decode_workspace_bytes(self.handle, self.case.B, self.max_seq_len, num_splits)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=self.v_pool.device)
        return self.workspace

    @property
    def max_seq_len(self) -> int:
        return int(self.case.seq_lens.max()) if self.case.B else 0

    def absorb(self) -> torch.Tensor:
        gb.gva_absorb_query(self.handle, self.q_c, self.q_r, self.M, self.q_pos, self.q_abs, self.case.B)
        return self.q_abs

    def append(self) -> None:
        gb.gva_append_cache(self.handle, self.cache, self.v_new, self.kr_new, self.append_pos, self.case.B,
                            self.status)

    def decode(self, num_splits: int = 0, q_abs: Optional[torch.Tensor] = None, seq_lens=None,
               max_seq_len: Optional[int] = None):
        ws = self.ensure_workspace(num_splits)
        gb.gva_decode(self.handle, self.cache, self.q_abs if q_abs is None else q_abs,
                      self.seq_lens if seq_lens is None else seq_lens, self.out, self.lse, ws, self.case.B,
                      self.max_seq_len if max_seq_len is None else max_seq_len, num_splits, self.status)
        return self.out, self.lse

    def step(self, num_splits: int = 0):
        """absorb + append + decode through the fused entry point (append position = query position)."""
        ws = self.ensure_workspace(num_splits)
        gb.gva_decode_step(self.handle, self.cache, self.M, self.q_c, self.q_r, self.v_new, self.kr_new, self.append_pos,
                           self.seq_lens, self.q_abs, self.out, self.lse, ws, self.case.B, self.max_seq_len, num_splits,
                           self.status)
        return self.out, self.lse

    def pools_to_host(self):
        v = self.v_pool.cpu().numpy()
        k = self.kr_pool.cpu().numpy()
        if self.case.cache_dtype == "bf16":
            v, k = v.view(np.uint16), k.view(np.uint16)
        return v, k

    def close(self) -> None:
        if self.handle:
            gb.gva_destroy(self.handle)
            self.handle = 0


def upload(case: DecodeCase, device="cuda:0", kernel: int = gb.GVA_KERNEL_AUTO) -> DeviceCase:
    dev = torch.device(device)
    s = case.shape
    handle = gb.gva_create(H=s.H, G=s.G, d_v=s.d_v, d_c=s.d_c, d_r=s.d_r, page_size=case.page_size,
                           cache_dtype={"bf16": gb.GVA_BF16, "fp8": gb.GVA_E4M3}.get(case.cache_dtype, gb.GVA_F32), kernel=kernel,
                           rope_base=case.rope_base, device=dev.index or 0)
    B = case.B
    return DeviceCase(
        case=case, handle=handle, v_pool=_dev(case.v_pool, dev), kr_pool=_dev(case.kr_pool, dev),
        block_table=_dev(case.block_table, dev), seq_lens=_dev(case.seq_lens, dev), q_c=_dev(case.q_c, dev),
        q_r=_dev(case.q_r, dev), M=_dev(case.M, dev), q_pos=_dev(case.q_pos, dev), v_new=_dev(case.v_new, dev),
        kr_new=_dev(case.kr_new, dev), append_pos=_dev(case.append_pos, dev),
        q_abs=torch.empty((B, s.H, s.d_v + s.d_r), dtype=torch.float32, device=dev),
        out=torch.full((B, s.H, s.d_v), float("nan"), dtype=torch.float32, device=dev),
        lse=torch.full((B, s.H), float("nan"), dtype=torch.float32, device=dev),
        status=torch.zeros(1, dtype=torch.int32, device=dev))


@dataclass
class GqaDeviceCase:
    """Matched GQA decode inputs on the device (from workloads.gqa_case)."""
    g: dict
    handle: int
    k_pool: torch.Tensor
    v_pool: torch.Tensor
    block_table: Optional[torch.Tensor]
    seq_lens: torch.Tensor
    q: torch.Tensor
    out: torch.Tensor
    lse: torch.Tensor
    status: torch.Tensor
    workspace: Optional[torch.Tensor] = None

    @property
    def cache(self) -> gb.GqaCache:
        return gb.make_gqa_cache(self.k_pool, self.v_pool, self.block_table, self.g["num_pages"],
                                 self.g["max_pages_per_seq"])

    def decode(self, num_splits: int = 0):
        B = self.g["B"]
        max_len = int(self.g["seq_lens"].max()) if B else 0
        need = gb.gva_decode_workspace_bytes(self.handle, B, max_len, num_splits)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=self.q.device)
        gb.gqa_decode(self.handle, self.cache, self.q, self.seq_lens, self.out, self.lse, self.workspace, B, max_len,
                      num_splits, self.status)
        return self.out, self.lse

    def close(self) -> None:
        if self.handle:
            gb.gva_destroy(self.handle)
            self.handle = 0


def upload_gqa(g: dict, device="cuda:0", kernel: int = gb.GVA_KERNEL_AUTO) -> GqaDeviceCase:
    dev = torch.device(device)
    d_h = g["d_h"]
    handle = gb.gva_create(H=g["H"], G=g["G"], d_v=d_h, d_c=d_h, d_r=16 if d_h == 64 else 32, page_size=g["page_size"],
                           cache_dtype={"bf16": gb.GVA_BF16, "fp8": gb.GVA_E4M3}.get(g["cache_dtype"], gb.GVA_F32), kernel=kernel,
                           device=dev.index or 0)
    B = g["B"]
    return GqaDeviceCase(g=g, handle=handle, k_pool=_dev(g["k_pool"], dev), v_pool=_dev(g["v_pool"], dev),
                         block_table=_dev(g["block_table"], dev), seq_lens=_dev(g["seq_lens"], dev), q=_dev(g["q"], dev),
                         out=torch.full((B, g["H"], d_h), float("nan"), dtype=torch.float32, device=dev),
                         lse=torch.full((B, g["H"]), float("nan"), dtype=torch.float32, device=dev),
                         status=torch.zeros(1, dtype=torch.int32, device=dev))


@dataclass
class PrefillDeviceCase:
    """A workloads.PrefillCase on the device: the cache (through a DeviceCase) plus the chunk's per-token tensors."""
    pc: object
    dc: DeviceCase
    cu_q: torch.Tensor
    ctx_lens: torch.Tensor
    q_c: torch.Tensor
    q_r: torch.Tensor
    q_pos: torch.Tensor
    v_new: torch.Tensor
    kr_new: torch.Tensor
    q_abs: torch.Tensor
    out: torch.Tensor
    lse: torch.Tensor
    _ws: Optional[torch.Tensor] = None

    @property
    def handle(self) -> int:
        return self.dc.handle

    @property
    def status(self) -> torch.Tensor:
        return self.dc.status

    @property
    def max_q_len(self) -> int:
        return int(self.pc.q_lens.max()) if len(self.pc.q_lens) else 0

    def absorb(self) -> torch.Tensor:
        gb.gva_absorb_query(self.handle, self.q_c, self.q_r, self.dc.M, self.q_pos, self.q_abs, self.pc.n_q)
        return self.q_abs

    def append(self) -> None:
        gb.gva_append_chunk(self.handle, self.dc.cache, self.v_new, self.kr_new, self.cu_q, self.ctx_lens, self.pc.cache.B,
                            self.pc.n_q, self.status)

    def prefill(self, max_q_len: Optional[int] = None):
        gb.gva_prefill(self.handle, self.dc.cache, self.q_abs, self.cu_q, self.ctx_lens, self.out, self.lse, self.pc.cache.B,
                       self.max_q_len if max_q_len is None else max_q_len, self.status)
        return self.out, self.lse

    def decode_multi(self, num_splits: int = 0):
        """The same attention with split-KV (gva_decode_multi): for few new tokens over a long cached context."""
        c = self.pc.cache
        max_len = int(c.seq_lens.max()) if c.B else 0
        need = gb.gva_decode_multi_workspace_bytes(self.handle, c.B, self.pc.n_q, self.max_q_len, max_len, num_splits)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=self.q_abs.device)
        gb.gva_decode_multi(self.handle, self.dc.cache, self.q_abs, self.cu_q, self.ctx_lens, self.out, self.lse, ws, c.B,
                            self.pc.n_q, self.max_q_len, max_len, num_splits, self.status)
        self._ws = ws          # keep the workspace alive until the stream has run
        return self.out, self.lse

    def decode_tokens(self, q_len: int, num_splits: int = 0):
        """The same attention for exactly q_len new tokens per sequence on the split-KV decode kernel (gva_decode_tokens)."""
        c = self.pc.cache
        max_len = int(c.seq_lens.max()) if c.B else 0
        need = gb.gva_decode_tokens_workspace_bytes(self.handle, c.B, q_len, max_len, num_splits)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=self.q_abs.device)
        gb.gva_decode_tokens(self.handle, self.dc.cache, self.q_abs, self.dc.seq_lens, self.out, self.lse, ws, c.B, q_len, max_len,
                             num_splits, self.status)
        self._ws = ws
        return self.out, self.lse

    def decode_tokens_ragged(self, num_splits: int = 0):
        """The same with every sequence's own number of new tokens (at most 8): gva_decode_tokens_ragged."""
        c = self.pc.cache
        max_len = int(c.seq_lens.max()) if c.B else 0
        mq = max(self.max_q_len, 1)
        need = gb.gva_decode_tokens_workspace_bytes(self.handle, c.B, max(mq, 2), max_len, num_splits)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=self.q_abs.device)
        gb.gva_decode_tokens_ragged(self.handle, self.dc.cache, self.q_abs, self.cu_q, self.dc.seq_lens, self.out, self.lse, ws,
                                    c.B, mq, max_len, num_splits, self.status)
        self._ws = ws
        return self.out, self.lse

    def close(self) -> None:
        self.dc.close()


def upload_prefill(pc, device="cuda:0") -> PrefillDeviceCase:
    dev = torch.device(device)
    dc = upload(pc.cache, device=device)
    s = pc.cache.shape
    n = pc.n_q
    return PrefillDeviceCase(
        pc=pc, dc=dc, cu_q=_dev(pc.cu_q, dev), ctx_lens=_dev(pc.ctx_lens, dev), q_c=_dev(pc.q_c, dev), q_r=_dev(pc.q_r, dev),
        q_pos=_dev(pc.q_pos, dev), v_new=_dev(pc.v_new, dev), kr_new=_dev(pc.kr_new, dev),
        q_abs=torch.empty((max(n, 1), s.H, s.d_v + s.d_r), dtype=torch.float32, device=dev),
        out=torch.full((max(n, 1), s.H, s.d_v), float("nan"), dtype=torch.float32, device=dev),
        lse=torch.full((max(n, 1), s.H), float("nan"), dtype=torch.float32, device=dev))
