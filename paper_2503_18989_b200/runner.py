"""Device-side driver for a workload scenario: owns the torch buffers and calls the C-ABI library.

PyTorch is used here for device memory and streams only; every step of the path
(plan, append, attention, merge) runs inside libhat.so through `binding`.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from .workloads import CacheSpec, Scenario, Step


def _dev_u16(a: np.ndarray, device) -> torch.Tensor:
    """uint16 bit patterns -> device tensor (stored as int16; only the bits matter)."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device, non_blocking=False)


_GUARD_BYTES = 1024      # canary zone in front of and behind every buffer the library writes
_GUARD_BYTE = 0x5A


class _Guarded:
    """A device buffer between two canary zones: `view` is what the library gets, intact() tells whether anything
    was written outside it."""

    def __init__(self, shape, dtype, fill, device):
        n = 1
        for x in shape:
            n *= int(x)
        item = torch.empty(0, dtype=dtype).element_size()
        self.nbytes = n * item
        pad = (-self.nbytes) % 256                       # keep the rear zone (and the next allocation) aligned
        self.raw = torch.full((_GUARD_BYTES + self.nbytes + pad + _GUARD_BYTES,), _GUARD_BYTE, dtype=torch.uint8, device=device)
        self.view = self.raw[_GUARD_BYTES:_GUARD_BYTES + self.nbytes].view(dtype).view(*shape)
        if fill is not None:
            self.view.fill_(fill)

    def intact(self) -> bool:
        front = self.raw[:_GUARD_BYTES]
        rear = self.raw[_GUARD_BYTES + self.nbytes:]
        return bool((front == _GUARD_BYTE).all().item()) and bool((rear == _GUARD_BYTE).all().item())


class DeviceCache:
    """K and V pools of one layer on the device."""

    def __init__(self, spec: CacheSpec, k_pool: np.ndarray, v_pool: np.ndarray, device="cuda:0"):
        self.spec = spec
        self.device = torch.device(device)
        self.k = _dev_u16(k_pool, self.device)
        self.v = _dev_u16(v_pool, self.device)
        self.desc = B.make_cache_desc(spec.dtype, spec.num_pages, spec.num_heads, spec.head_dim,
                                      spec.stride_page, spec.stride_token, spec.stride_head, self.k, self.v,
                                      spec.page_size)

    def pools_to_host(self):
        return (self.k.cpu().numpy().view(np.uint16), self.v.cpu().numpy().view(np.uint16))


class DeviceStep:
    """One batch resident on the device, with its plan, outputs and workspace."""

    def __init__(self, cache: DeviceCache, step: Step):
        dev = cache.device
        spec = cache.spec
        self.cache = cache
        self.step = step
        H = int(step.q.shape[1])                  # query heads; spec.num_heads K/V heads
        self.plan = B.hat_plan_create(cache.desc, H, step.cu_chunk, step.prefix_len, step.chunk_len,
                                      step.block_table, tree_mask=getattr(step, "tree_mask", None))
        self.info = B.hat_plan_get_info(self.plan).as_dict()
        T, d = step.total_rows, spec.head_dim
        self.q = _dev_u16(step.q, dev)
        self.k_new = _dev_u16(step.k_new, dev)
        self.v_new = _dev_u16(step.v_new, dev)
        # every buffer the library writes sits between canary zones (checked by canaries_intact)
        self._g_out = _Guarded((T, H, d), torch.float32, float("nan"), dev)
        self._g_lse = _Guarded((T, H), torch.float32, float("nan"), dev)
        self.out, self.lse = self._g_out.view, self._g_lse.view
        self.workspace_bytes = B.hat_plan_workspace_bytes(self.plan)
        self._g_ws = _Guarded((max(self.workspace_bytes, 256),), torch.uint8, None, dev)
        self.workspace = self._g_ws.view
        self._g_out16 = None

    def append(self, stream: int = 0) -> None:
        B.hat_kv_append(self.cache.desc, self.plan, self.k_new, self.v_new, stream)

    def attend16(self, fused_append: bool = True, sm_scale: float = 0.0, stream: int = 0) -> None:
        """The same step with the output in the cache's 16-bit type (self.out16, allocated on first use)."""
        if getattr(self, "out16", None) is None:
            self._g_out16 = _Guarded(tuple(self.out.shape), torch.int16, -1, self.out.device)
            self.out16 = self._g_out16.view
        B.hat_chunk_attention_out16(self.cache.desc, self.plan, self.q,
                                    self.k_new if fused_append else None, self.v_new if fused_append else None,
                                    self.out16, self.lse, sm_scale, self.workspace, self.workspace_bytes, stream)

    def attend(self, fused_append: bool = True, sm_scale: float = 0.0, stream: int = 0) -> None:
        B.hat_chunk_attention(self.cache.desc, self.plan, self.q,
                              self.k_new if fused_append else None, self.v_new if fused_append else None,
                              self.out, self.lse, sm_scale, self.workspace, self.workspace_bytes, stream)

    def results(self):
        torch.cuda.synchronize(self.cache.device)
        return self.out.cpu().numpy(), self.lse.cpu().numpy()

    def canaries_intact(self) -> bool:
        """No byte outside out / lse / workspace (/ out16) was written."""
        torch.cuda.synchronize(self.cache.device)
        return all(g.intact() for g in (self._g_out, self._g_lse, self._g_ws, self._g_out16) if g is not None)

    def close(self):
        self.plan.close()


def run_scenario(sc: Scenario, device="cuda:0", fused_append: bool = True):
    """Run every step of a scenario in order; returns (cache, [(out, lse) per step])."""
    cache = DeviceCache(sc.cache, sc.k_pool, sc.v_pool, device)
    res = []
    for st in sc.steps:
        ds = DeviceStep(cache, st)
        if not fused_append:
            ds.append()
        ds.attend(fused_append=fused_append)
        res.append(ds.results())
        status = B.hat_last_device_status(ds.plan)
        if status != B.HAT_OK:
            raise RuntimeError(f"device status {status}: {B.hat_status_string(status)}")
        if not ds.canaries_intact():
            raise RuntimeError("a canary zone around out / lse / workspace was overwritten")
        ds.close()
    return cache, res
