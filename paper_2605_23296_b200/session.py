"""Device-buffer bookkeeping around the C-ABI calls for one compaction event.

PyTorch is used for device memory and streams only; every step of the path
(planning, prefill, append, decode, merge) runs inside libcompact_attn.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as B


def bits_to_tensor(bits: np.ndarray, device=None, pin: bool = False) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor (same bits)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if pin:
        t = t.pin_memory()
    return t.to(device, non_blocking=pin) if device is not None else t


def tensor_to_bits(t: torch.Tensor) -> np.ndarray:
    """torch.bfloat16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class CompactionSession:
    """One history cut into blocks, one summary sequence per block (paper, Section 4).

    Owns the plan handle, the device index buffer, the K/V page pools and the
    decode workspace.  All calls are enqueued on the current torch stream of
    `device` unless a stream is given.
    """

    def __init__(self, block_lens: Sequence[int], max_new_tokens: int, num_q_heads: int,
                 num_kv_heads: int, head_dim: int, free_pages: Sequence[int], num_pages: int,
                 scale: Optional[float] = None, device: str = "cuda:0", pages_per_split: int = 0,
                 poison_pools: bool = False, page_size: int = 16, q_tile_rows: int = 0,
                 prefix_lens: Optional[Sequence[int]] = None, shared_pages: Optional[Sequence[int]] = None,
                 pools=None, num_sms: int = 0, chunk_tokens: int = 0, decode_sms: int = 0, dynamic_pages: bool = False,
                 decode_steps_per_chunk: int = 1):
        self.device = torch.device(device)
        self.Hq, self.Hkv, self.d, self.P = num_q_heads, num_kv_heads, head_dim, page_size
        self.B = len(block_lens)
        self.block_lens = np.asarray(block_lens, dtype=np.int32)
        self.scale = float(scale if scale is not None else head_dim ** -0.5)
        props = torch.cuda.get_device_properties(self.device)
        # num_sms is the SM budget of this event: the persistent prefill grid and the decode wave are sized
        # from it (all SMs unless the caller wants to leave room for other work on the device)
        self.cfg = B.cpa_config(num_q_heads, num_kv_heads, head_dim, page_size, self.scale, q_tile_rows,
                                pages_per_split, num_sms or props.multi_processor_count)
        self.prefix_aware = prefix_lens is not None
        self.chunk_tokens = chunk_tokens
        self.dynamic_pages = dynamic_pages
        if dynamic_pages:       # no pages reserved for the summaries: blocks draw from a common reserve as they grow
            assert prefix_lens is None and not chunk_tokens
            self.plan = B.cpa_plan_create_dynamic(self.cfg, self.block_lens, max_new_tokens, free_pages)
        elif chunk_tokens and self.prefix_aware:   # both: cached history prefix, own tokens in chunks
            self.plan = B.cpa_plan_create_prefix_chunked(self.cfg, self.block_lens, prefix_lens, shared_pages,
                                                         max_new_tokens, chunk_tokens, free_pages, decode_sms,
                                                         decode_steps_per_chunk)
        elif chunk_tokens:      # prefill in chunks, mixed with the decode of blocks that are past their prompt
            self.plan = B.cpa_plan_create_chunked(self.cfg, self.block_lens, max_new_tokens, chunk_tokens, free_pages,
                                                  decode_sms, decode_steps_per_chunk)
        elif self.prefix_aware:   # the paper's layout: cached history prefix + own tokens per worker
            self.plan = B.cpa_plan_create_prefix(self.cfg, self.block_lens, prefix_lens, shared_pages,
                                                 max_new_tokens, free_pages)
        else:
            self.plan = B.cpa_plan_create(self.cfg, self.block_lens, max_new_tokens, free_pages)
        self.total_tokens = B.cpa_plan_param(self.plan, B.PARAM_TOTAL_TOKENS)
        nbytes = B.cpa_plan_param(self.plan, B.PARAM_INDEX_BYTES)
        self.index_buf = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        pool_shape = (num_pages, num_kv_heads, page_size, head_dim)
        if pools is not None:   # pools that already hold a cached history (shared with another session)
            self.k_pool, self.v_pool = pools
            assert tuple(self.k_pool.shape) == pool_shape and tuple(self.v_pool.shape) == pool_shape
        elif poison_pools:   # unused slots hold NaN: the kernels must mask by index, not by value
            self.k_pool = torch.full(pool_shape, float("nan"), dtype=torch.bfloat16, device=self.device)
            self.v_pool = torch.full(pool_shape, float("nan"), dtype=torch.bfloat16, device=self.device)
        else:  # no initialisation needed: slots are masked by index until they are written
            self.k_pool = torch.empty(pool_shape, dtype=torch.bfloat16, device=self.device)
            self.v_pool = torch.empty(pool_shape, dtype=torch.bfloat16, device=self.device)
        ws = B.cpa_plan_param(self.plan, B.PARAM_DECODE_WORKSPACE_BYTES)
        self.workspace = torch.empty(max(ws, 256), dtype=torch.uint8, device=self.device)
        self._check(B.cpa_plan_upload(self.plan, self.index_buf, nbytes, self._stream()), "cpa_plan_upload")

    # -- helpers ------------------------------------------------------------
    def _stream(self) -> int:
        return int(torch.cuda.current_stream(self.device).cuda_stream)

    @staticmethod
    def _check(rc: int, where: str) -> None:
        if rc != B.CPA_OK:
            raise B.CpaError(rc, where)

    def export(self, which: int) -> np.ndarray:
        return B.cpa_plan_export(self.plan, which)

    def param(self, which: int) -> int:
        return B.cpa_plan_param(self.plan, which)

    # -- the hot path -------------------------------------------------------
    def prefill(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                out: Optional[torch.Tensor] = None, variant: Optional[int] = None) -> torch.Tensor:
        """Causal attention of every block over itself; q/out [tokens,Hq,d], k/v [tokens,Hkv,d]."""
        if out is None:
            out = torch.empty_like(q)
        if self.prefix_aware:
            self._check(B.cpa_prefill_prefix(self.plan, q, k, v, self.k_pool, self.v_pool, out, self._stream()),
                        "cpa_prefill_prefix")
        elif variant is None:
            self._check(B.cpa_prefill(self.plan, q, k, v, out, None, self._stream()), "cpa_prefill")
        else:
            self._check(B.cpa_prefill_variant(self.plan, q, k, v, out, self._stream(), variant),
                        "cpa_prefill_variant")
        return out

    def append_prefill(self, k: torch.Tensor, v: torch.Tensor) -> None:
        """Store the prefill K/V of every block in its pages."""
        self._check(B.cpa_kv_append(self.plan, k, v, self.block_lens, self.k_pool, self.v_pool,
                                    self._stream()), "cpa_kv_append")

    def append(self, k_new: torch.Tensor, v_new: torch.Tensor, new_lens=None) -> None:
        """One token per block (new_lens None) or new_lens[b] tokens per block."""
        self._check(B.cpa_kv_append(self.plan, k_new, v_new, new_lens, self.k_pool, self.v_pool,
                                    self._stream()), "cpa_kv_append")

    def decode(self, q: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q/out [B,Hq,d]: newest token of every block over that block's cache."""
        if out is None:
            out = torch.empty_like(q)
        self._check(B.cpa_decode(self.plan, q, self.k_pool, self.v_pool, out, self.workspace,
                                 self._stream()), "cpa_decode")
        return out

    def decode_append(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """One decode step with its append fused in (same result as append() then decode())."""
        if out is None:
            out = torch.empty_like(q)
        self._check(B.cpa_decode_append(self.plan, q, k_new, v_new, self.k_pool, self.v_pool, out,
                                        self.workspace, self._stream()), "cpa_decode_append")
        return out

    def decode_append_steps(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                            out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q/out [n,B,Hq,d], k_new/v_new [n,B,Hkv,d]: n consecutive fused decode steps enqueued by one call."""
        if out is None:
            out = torch.empty_like(q)
        assert q.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous() and out.is_contiguous()
        self._check(B.cpa_decode_append_steps(self.plan, q, k_new, v_new, self.k_pool, self.v_pool, out,
                                              self.workspace, q.shape[0], self._stream()), "cpa_decode_append_steps")
        return out

    def step_mixed(self, step: int, q, k, v, out, q_dec=None, k_new=None, v_new=None, out_dec=None) -> None:
        """Step `step` of a chunked plan: the chunk that starts at this step, if any (rows of the whole-event
        tensors q/k/v/out), beside one decode token of the blocks whose turn it is."""
        self._check(B.cpa_step_mixed(self.plan, step, q, k, v, out, q_dec, k_new, v_new, out_dec, self.k_pool,
                                     self.v_pool, self.workspace, self._stream()), "cpa_step_mixed")

    def event_from_host(self, h_q, h_k, h_v, h_out, h_q_dec=None, h_k_dec=None, h_v_dec=None, h_out_dec=None,
                        stage: Optional[torch.Tensor] = None) -> torch.Tensor:
        """The whole event from host tensors (page-locked ones overlap with the kernels): prompts [tokens,H,d],
        decode steps' inputs [T,B,H,d]; h_out / h_out_dec are written.  Everything is enqueued on the current
        stream; synchronise it before reading the outputs.  Returns the device staging buffer (uint8,
        PARAM_HOST_STAGE_BYTES), which a later event of the same shape may be given again."""
        need = self.param(B.PARAM_HOST_STAGE_BYTES)
        if stage is None:
            stage = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
        assert stage.numel() >= need and stage.device == self.device
        self._check(B.cpa_event_host(self.plan, h_q, h_k, h_v, h_out, h_q_dec, h_k_dec, h_v_dec, h_out_dec, stage,
                                     self.k_pool, self.v_pool, self.workspace, self._stream()), "cpa_event_host")
        return stage

    def step_mixed_range(self, first_step: int, num_steps: int, q, k, v, out, q_dec=None, k_new=None, v_new=None,
                         out_dec=None) -> None:
        """Steps first_step .. first_step + num_steps - 1 of a chunked plan by one call; the decode tensors are
        [num_steps, B, H, d], slice i for step first_step + i."""
        self._check(B.cpa_step_mixed_range(self.plan, first_step, num_steps, q, k, v, out, q_dec, k_new, v_new,
                                           out_dec, self.k_pool, self.v_pool, self.workspace, self._stream()),
                    "cpa_step_mixed_range")

    def decode_append_dynamic(self, q, k_new, v_new, active=None, out=None):
        """One decode step of a plan with pages on demand; `active` is a device int32 [B] tensor of stop flags."""
        if out is None:
            out = torch.empty_like(q)
        self._check(B.cpa_decode_append_dynamic(self.plan, q, k_new, v_new, active, self.k_pool, self.v_pool, out,
                                                self.workspace, self._stream()), "cpa_decode_append_dynamic")
        return out

    def release(self, active) -> None:
        """Blocks whose flag is 0 give their pages back to the reserve."""
        self._check(B.cpa_release_blocks(self.plan, active, self._stream()), "cpa_release_blocks")

    def sync(self) -> None:
        """Read the device's lengths, page table and reserve back into the plan's host copies."""
        self._check(B.cpa_plan_sync(self.plan, self._stream()), "cpa_plan_sync")

    def status(self) -> int:
        return B.cpa_plan_status(self.plan, self._stream())

    def close(self) -> None:
        if self.plan:
            torch.cuda.synchronize(self.device)
            B.cpa_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass
