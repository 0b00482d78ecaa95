"""Convenience layer for tests and the benchmark: device buffers (torch) around the C-ABI calls.

Nothing here computes anything about grammars or masks; it allocates tensors, passes their
pointers through `binding`, and moves results to numpy.  It needs a CUDA device.
"""
from __future__ import annotations

import os
import time
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from . import inputs


class Session:
    """One tokenizer, its compiled grammars and one matcher per request of a workload."""

    def __init__(self, workload: inputs.Workload, share_pool: bool = True, device: str = "cuda:0", state_compression: bool = True,
                 jit: bool = False, jit_precompute: int = 0, jit_arena_bytes: int = 0, compile_threads: int = 0,
                 reserve_bytes: int = 0, repeat_threshold: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU path)")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.w = workload
        v = workload.vocab
        self.tokenizer = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
        self.pool = B.CachePool(self.tokenizer) if share_pool else None
        if self.pool and reserve_bytes > 0:
            self.pool.reserve(reserve_bytes)       # device memory for the cache taken before the (timed) compiles
        # xg_compile_grammar may be called from several threads: the host front ends run side by side, the
        # cache builds take turns on the pool.  compile_threads: 0 = one per core (at most 16), 1 = in this thread.
        def compile_one(g):
            torch.cuda.set_device(self.device)
            return B.Grammar(self.tokenizer, g.kind, g.text, pool=self.pool, state_compression=state_compression,
                             jit=jit, jit_precompute=jit_precompute, jit_arena_bytes=jit_arena_bytes, repeat_threshold=repeat_threshold)
        n_threads = compile_threads if compile_threads > 0 else min(16, os.cpu_count() or 1)
        n_threads = max(1, min(n_threads, len(workload.grammars)))
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        if n_threads == 1:
            self.grammars: List[B.Grammar] = [compile_one(g) for g in workload.grammars]
        else:
            with ThreadPoolExecutor(max_workers=n_threads) as ex:
                self.grammars = list(ex.map(compile_one, workload.grammars))
        torch.cuda.synchronize()
        self.compile_wall_s = time.perf_counter() - t0       # the grammar compiles alone (tokenizer and matchers excluded)
        self.matchers = [B.Matcher(self.grammars[gi]) for gi in workload.request_grammar]
        self.batch = B.Batch(self.matchers)
        self.V, self.W, self.n = v.size, self.tokenizer.words, len(self.matchers)
        self.bitmask = torch.zeros((self.n, self.W), dtype=torch.int32, device=self.device)
        self.status = torch.zeros(self.n, dtype=torch.int32, device=self.device)
        self.accept_status = torch.zeros(self.n, dtype=torch.int32, device=self.device)
        self.tokens = torch.zeros(self.n, dtype=torch.int32, device=self.device)

    def stream(self) -> int:
        return torch.cuda.current_stream().cuda_stream

    def fill(self) -> None:
        self.batch.fill_next_token_bitmask(self.bitmask.data_ptr(), self.W, self.status.data_ptr(), self.stream())

    def accept(self, token_ids: Sequence[int], restart_on_eos: bool = False) -> None:
        self.tokens.copy_(torch.as_tensor(np.asarray(token_ids, dtype=np.int32)))
        self.batch.accept_token(self.tokens.data_ptr(), self.accept_status.data_ptr(), self.stream(), restart_on_eos)

    def accept_device(self, token_ids: torch.Tensor, restart_on_eos: bool = False) -> None:
        self.batch.accept_token(token_ids.data_ptr(), self.accept_status.data_ptr(), self.stream(), restart_on_eos)

    def accept_fill(self, token_ids: Sequence[int], restart_on_eos: bool = False) -> None:
        self.tokens.copy_(torch.as_tensor(np.asarray(token_ids, dtype=np.int32)))
        self.accept_fill_device(self.tokens, restart_on_eos)

    def accept_fill_device(self, token_ids: torch.Tensor, restart_on_eos: bool = False) -> None:
        """Accept one token per request and fill the next step's mask, in one launch."""
        self.batch.accept_token_and_fill_next_bitmask(token_ids.data_ptr(), self.accept_status.data_ptr(), restart_on_eos,
                                                      self.bitmask.data_ptr(), self.W, self.status.data_ptr(), self.stream())

    def apply(self, logits: torch.Tensor, rows: Optional[torch.Tensor] = None) -> None:
        dtype = {torch.float32: "f32", torch.bfloat16: "bf16", torch.int16: "bf16", torch.uint16: "bf16"}[logits.dtype]
        B.apply_token_bitmask(logits.data_ptr(), dtype, logits.shape[0], self.V, logits.stride(0), self.bitmask.data_ptr(), self.W,
                              rows.data_ptr() if rows is not None else 0, int(rows.numel()) if rows is not None else 0, self.stream())

    def fill_apply(self, logits: torch.Tensor) -> None:
        """Fill every request's mask and apply it to its logits row, in one launch."""
        dtype = {torch.float32: "f32", torch.bfloat16: "bf16", torch.int16: "bf16", torch.uint16: "bf16"}[logits.dtype]
        self.batch.fill_and_apply_token_bitmask(self.bitmask.data_ptr(), self.W, self.status.data_ptr(), logits.data_ptr(), dtype,
                                                logits.stride(0), self.stream())

    def jit_service(self, wait: bool = False) -> dict:
        """Between decode steps: pick up the cache entries the last fills found missing (just-in-time grammars)."""
        return B.jit_service(self.grammars, self.stream(), wait)

    def mask_numpy(self) -> np.ndarray:
        return self.bitmask.cpu().numpy().view(np.uint32)

    def reset(self, request: int) -> None:
        self.matchers[request].reset(self.stream())

    def close(self) -> None:
        torch.cuda.synchronize()
        for m in self.matchers:
            m.close()
        for g in self.grammars:
            g.close()
        if self.pool:
            self.pool.close()
        self.tokenizer.close()


def logits_tensor(arr: np.ndarray, device) -> torch.Tensor:
    """float32 array -> float32 tensor; uint16 bf16 bit patterns -> bfloat16 tensor."""
    if arr.dtype == np.float32:
        return torch.from_numpy(arr).to(device)
    return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)


def logits_numpy(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.float32:
        return t.cpu().numpy()
    return t.view(torch.int16).cpu().numpy().view(np.uint16)
