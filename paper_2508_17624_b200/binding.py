"""ctypes binding over libexpertweave.so: argument marshalling only.

Function names mirror the C ABI (`include/expertweave.h`).  Host weights are numpy uint16 arrays of
bf16 bit patterns; device operands are torch CUDA tensors, passed by data pointer together with the
current CUDA stream.  There is no CPU fallback: if the library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libexpertweave.so")

EW_OK = 0
STATUS_NAMES = ["EW_OK", "EW_ERR_INVALID_ARG", "EW_ERR_OOM", "EW_ERR_SLOT_IN_USE", "EW_ERR_NOT_LOADED",
                "EW_ERR_TOO_MANY_EXPERTS", "EW_ERR_CUDA", "EW_ERR_TIMEOUT", "EW_ERR_BAD_ADAPTER_ID_IN_BATCH",
                "EW_ERR_NO_DEVICE"]
EXPORTS = ["ew_pool_create", "ew_pool_destroy", "ew_load_base", "ew_load_adapter", "ew_unload_adapter",
           "ew_pool_trim", "ew_moe_forward", "ew_moe_forward_debug", "ew_moe_forward_host", "ew_profile_enable",
           "ew_profile_read", "ew_reroute", "ew_reroute_unfused", "ew_route_logits", "ew_route_noalloc", "ew_selftest_bounded_wait", "ew_get_expert_map",
           "ew_moe_forward_partial", "ew_ep_finish", "ew_moe_forward_scatter", "ew_ep_finish_gathered", "ew_pool_stats", "ew_last_device_error", "ew_slot_address", "ew_status_str", "ew_last_error_string"]


class EwConfig(C.Structure):
    _fields_ = [("device", C.c_int32), ("num_layers", C.c_int32), ("hidden", C.c_int32), ("inter", C.c_int32),
                ("num_experts", C.c_int32), ("num_shared", C.c_int32), ("top_k", C.c_int32),
                ("max_adapters", C.c_int32), ("e_max", C.c_int32), ("max_tokens", C.c_int32),
                ("renormalize", C.c_int32), ("routed_scale", C.c_float), ("pool_mode", C.c_int32),
                ("ep_size", C.c_int32), ("page_bytes", C.c_uint64), ("prealloc_pages", C.c_uint64),
                ("max_pages", C.c_uint64), ("ep_rank", C.c_int32), ("reserved0", C.c_int32)]


class EwStats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in
                ("page_bytes", "va_reserved_bytes", "pages_mapped", "pages_free", "pages_created_total",
                 "physical_bytes", "live_expert_bytes", "padding_bytes", "live_experts", "adapters_loaded",
                 "workspace_bytes", "last_forward_kernels")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class EwError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail else ""))


_lib = None


def lib():
    """Load the shared library (raises if it has not been built: there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2508_17624_b200.build` "
                               "(the CUDA extension is required; there is no CPU fallback)")
        _lib = C.CDLL(LIB_PATH)
        _lib.ew_status_str.restype = C.c_char_p
        _lib.ew_last_error_string.restype = C.c_char_p
        for name in EXPORTS:
            getattr(_lib, name)
    return _lib


def _check(rc: int, where: str):
    if rc != EW_OK:
        detail = lib().ew_last_error_string().decode() if rc == 6 or rc == 2 or rc == 1 else ""
        raise EwError(rc, where, detail)


def _host(a, dtype=np.uint16) -> Optional[np.ndarray]:
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=dtype)


def _hp(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dp(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Pool:
    """Owner of one `ew_pool_t`.  Methods carry the names of the C entry points without the prefix."""

    def __init__(self, *, device: int = 0, num_layers: int = 1, hidden: int, inter: int, num_experts: int,
                 num_shared: int, top_k: int, max_adapters: int, e_max: int, max_tokens: int,
                 renormalize: int = 0, routed_scale: float = 1.0, pool_mode: int = 0, page_bytes: int = 0,
                 prealloc_pages: int = 0, max_pages: int = 0, ep_size: int = 0, ep_rank: int = 0):
        self.cfg = EwConfig(device, num_layers, hidden, inter, num_experts, num_shared, top_k, max_adapters,
                            e_max, max_tokens, renormalize, routed_scale, pool_mode, ep_size, page_bytes,
                            prealloc_pages, max_pages, ep_rank, 0)
        self._h = C.c_void_p()
        _check(lib().ew_pool_create(C.byref(self.cfg), C.byref(self._h)), "ew_pool_create")

    @classmethod
    def from_config(cls, cfg, *, device: int = 0, max_tokens: Optional[int] = None, **kw) -> "Pool":
        """`cfg` is a `workloads.MoEConfig`."""
        return cls(device=device, num_layers=cfg.num_layers, hidden=cfg.hidden, inter=cfg.inter,
                   num_experts=cfg.num_experts, num_shared=cfg.num_shared, top_k=cfg.top_k,
                   max_adapters=cfg.max_adapters, e_max=cfg.e_max, max_tokens=max_tokens or cfg.n_tokens, **kw)

    @property
    def num_slots(self) -> int:
        return self.cfg.num_experts + self.cfg.max_adapters * self.cfg.e_max

    def destroy(self):
        if self._h:
            _check(lib().ew_pool_destroy(self._h), "ew_pool_destroy")
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def load_base(self, layer, router_w, w_gate, w_up, w_down, sh_gate=None, sh_up=None, sh_down=None):
        arrs = [_host(a) for a in (router_w, w_gate, w_up, w_down, sh_gate, sh_up, sh_down)]
        _check(lib().ew_load_base(self._h, layer, *[_hp(a) for a in arrs]), "ew_load_base")

    def load_adapter(self, adapter_id, counts, expert_ids, w_gate, w_up, w_down):
        """Weights: numpy arrays of bf16 bit patterns (host), or torch tensors (host or device) taken as they are."""
        counts = _host(counts, np.int32)
        expert_ids = _host(expert_ids, np.int32)
        keep = [a if hasattr(a, "data_ptr") else _host(a) for a in (w_gate, w_up, w_down)]   # alive during the call
        g, u, d = [_dp(a) if hasattr(a, "data_ptr") else _hp(a) for a in keep]
        _check(lib().ew_load_adapter(self._h, adapter_id, _hp(counts), _hp(expert_ids), g, u, d), "ew_load_adapter")

    def unload_adapter(self, adapter_id):
        _check(lib().ew_unload_adapter(self._h, adapter_id), "ew_unload_adapter")

    def trim(self):
        _check(lib().ew_pool_trim(self._h), "ew_pool_trim")

    def moe_forward(self, layer, x, adapter_ids, out=None):
        import torch
        if out is None:
            out = torch.empty_like(x)
        _check(lib().ew_moe_forward(self._h, layer, _dp(x), _dp(adapter_ids), x.shape[0], _dp(out), _stream()),
               "ew_moe_forward")
        return out

    def moe_forward_partial(self, layer, x, adapter_ids, partial=None):
        """This rank's unrounded partial sums, fp32 [n_tokens, H] (expert parallelism; see the header)."""
        import torch
        if partial is None:
            partial = torch.empty(x.shape, dtype=torch.float32, device=x.device)
        _check(lib().ew_moe_forward_partial(self._h, layer, _dp(x), _dp(adapter_ids), x.shape[0], _dp(partial), _stream()),
               "ew_moe_forward_partial")
        return partial

    def ep_finish(self, summed, out=None):
        """bf16 result from the sum of all ranks' partials."""
        import torch
        if out is None:
            out = torch.empty(summed.shape, dtype=torch.bfloat16, device=summed.device)
        _check(lib().ew_ep_finish(self._h, _dp(summed), summed.shape[0], _dp(out), _stream()), "ew_ep_finish")
        return out

    def moe_forward_scatter(self, layer, x, adapter_ids, gather_ptrs):
        """Partial forward whose last kernel stores the partial sums into every rank's gather buffer; `gather_ptrs`:
        device int64 tensor with the ep_size buffer addresses (see the header)."""
        _check(lib().ew_moe_forward_scatter(self._h, layer, _dp(x), _dp(adapter_ids), x.shape[0], _dp(gather_ptrs), _stream()),
               "ew_moe_forward_scatter")

    def ep_finish_gathered(self, gathered, out=None):
        """bf16 result from this rank's gather buffer [ep_size, n_tokens, H] (blocks added in rank order)."""
        import torch
        if out is None:
            out = torch.empty(gathered.shape[1:], dtype=torch.bfloat16, device=gathered.device)
        _check(lib().ew_ep_finish_gathered(self._h, _dp(gathered), gathered.shape[1], _dp(out), _stream()), "ew_ep_finish_gathered")
        return out

    def moe_forward_debug(self, layer, x, adapter_ids):
        import torch
        B, k, P = x.shape[0], self.cfg.top_k, self.num_slots
        dev = x.device
        out = torch.empty_like(x)
        r = dict(topk_ids=torch.empty((B, k), dtype=torch.int32, device=dev),
                 topk_w=torch.empty((B, k), dtype=torch.float32, device=dev),
                 slot_ids=torch.empty((B, k), dtype=torch.int32, device=dev),
                 counts=torch.empty((P,), dtype=torch.int32, device=dev),
                 inv=torch.empty((B, k), dtype=torch.int32, device=dev),
                 offsets=torch.empty((P + 1,), dtype=torch.int32, device=dev))
        _check(lib().ew_moe_forward_debug(self._h, layer, _dp(x), _dp(adapter_ids), B, _dp(out), _stream(),
                                          _dp(r["topk_ids"]), _dp(r["topk_w"]), _dp(r["slot_ids"]), _dp(r["counts"]),
                                          _dp(r["inv"]), _dp(r["offsets"])), "ew_moe_forward_debug")
        r["out"] = out
        return r

    def moe_forward_host(self, layer, x_host, adapter_ids_host, out_host, n_tokens=None):
        """x_host / out_host: pinned torch CPU tensors (or numpy arrays); asynchronous on the current stream."""
        def hp(t):
            return C.c_void_p(t.data_ptr()) if hasattr(t, "data_ptr") else t.ctypes.data_as(C.c_void_p)
        n = x_host.shape[0] if n_tokens is None else n_tokens
        _check(lib().ew_moe_forward_host(self._h, layer, hp(x_host), hp(adapter_ids_host), n, hp(out_host),
                                         _stream()), "ew_moe_forward_host")
        return out_host

    def profile_enable(self, on: bool):
        _check(lib().ew_profile_enable(self._h, int(on)), "ew_profile_enable")

    def profile_read(self):
        """-> (dict kernel -> total ms, forwards measured)"""
        ms = (C.c_double * 5)()
        n = C.c_int32(0)
        _check(lib().ew_profile_read(self._h, ms, C.byref(n)), "ew_profile_read")
        names = ("route", "permute", "gemm1", "gemm2", "combine")
        return {k: float(v) for k, v in zip(names, ms)}, int(n.value)

    def reroute(self, layer, topk_ids, adapter_ids, slot_ids=None, counts=None, want_counts=True):
        import torch
        if slot_ids is None:
            slot_ids = torch.empty_like(topk_ids)
        if counts is None and want_counts:
            counts = torch.empty((self.num_slots,), dtype=torch.int32, device=topk_ids.device)
        _check(lib().ew_reroute(self._h, layer, _dp(topk_ids), _dp(adapter_ids), topk_ids.shape[0], _dp(slot_ids),
                                _dp(counts), _stream()), "ew_reroute")
        return slot_ids, counts

    def reroute_unfused(self, layer, topk_ids, adapter_ids, slot_ids=None, counts=None, want_counts=True, scratch=None):
        """The same rewrite as `reroute`, as one kernel per elementary tensor operation (ablation)."""
        import torch
        if slot_ids is None:
            slot_ids = torch.empty_like(topk_ids)
        if counts is None and want_counts:
            counts = torch.empty((self.num_slots,), dtype=torch.int32, device=topk_ids.device)
        if scratch is None:
            scratch = torch.empty((2 * topk_ids.numel(),), dtype=torch.int32, device=topk_ids.device)
        _check(lib().ew_reroute_unfused(self._h, layer, _dp(topk_ids), _dp(adapter_ids), topk_ids.shape[0], _dp(slot_ids),
                                        _dp(counts), _dp(scratch), _stream()), "ew_reroute_unfused")
        return slot_ids, counts

    def route_logits(self, layer, logits, adapter_ids):
        """Softmax + top-k + rerouting + per-slot counts from fp32 logits [n, M] (device tensors)."""
        import torch
        n, k, dev = logits.shape[0], self.cfg.top_k, logits.device
        ids = torch.empty((n, k), dtype=torch.int32, device=dev)
        w = torch.empty((n, k), dtype=torch.float32, device=dev)
        slots = torch.empty((n, k), dtype=torch.int32, device=dev)
        counts = torch.empty((self.num_slots,), dtype=torch.int32, device=dev)
        _check(lib().ew_route_logits(self._h, layer, _dp(logits), _dp(adapter_ids), n, _dp(ids), _dp(w), _dp(slots),
                                     _dp(counts), _stream()), "ew_route_logits")
        return ids, w, slots, counts

    def route_noalloc(self, layer, x, adapter_ids, topk_ids, topk_w, slot_ids, counts, device_status=None):
        """Routing into caller-provided device tensors; the library allocates nothing (see the header)."""
        _check(lib().ew_route_noalloc(self._h, layer, _dp(x), _dp(adapter_ids), x.shape[0], _dp(topk_ids),
                                      _dp(topk_w), _dp(slot_ids), _dp(counts), _dp(device_status), _stream()),
               "ew_route_noalloc")

    def selftest_bounded_wait(self):
        _check(lib().ew_selftest_bounded_wait(self._h, _stream()), "ew_selftest_bounded_wait")

    def get_expert_map(self, layer) -> np.ndarray:
        out = np.empty((self.cfg.max_adapters, self.cfg.num_experts), np.int32)
        _check(lib().ew_get_expert_map(self._h, layer, _hp(out)), "ew_get_expert_map")
        return out

    def stats(self) -> dict:
        s = EwStats()
        _check(lib().ew_pool_stats(self._h, C.byref(s)), "ew_pool_stats")
        return s.as_dict()

    def last_device_error(self) -> int:
        code = C.c_int32(0)
        _check(lib().ew_last_device_error(self._h, C.byref(code)), "ew_last_device_error")
        return code.value

    def slot_address(self, layer, which, slot) -> int:
        p = C.c_void_p()
        _check(lib().ew_slot_address(self._h, layer, which, slot, C.byref(p)), "ew_slot_address")
        return p.value or 0


def load_model(pool: Pool, cfg, bank=None, layers=None, adapters=None, tuned=None):
    """Fill a pool with the seeded synthetic model of `cfg` (a workloads.MoEConfig): base weights of the
    given layers, then the given adapters.  Returns (tuned sets, dict layer -> BaseLayer) for the tests."""
    from . import workloads as wl
    bank = bank or wl.NoiseBank(cfg.seed)
    layers = list(range(cfg.num_layers)) if layers is None else layers
    tuned = wl.tuned_sets(cfg) if tuned is None else tuned
    bases = {}
    for l in layers:
        b = wl.gen_base_layer(cfg, l, bank)
        pool.load_base(l, b.router_w, b.routed.w_gate, b.routed.w_up, b.routed.w_down,
                       b.shared.w_gate, b.shared.w_up, b.shared.w_down)
        bases[l] = b
    adapters = list(range(cfg.max_adapters)) if adapters is None else adapters
    for i in adapters:
        per_layer = [wl.gen_adapter_layer(cfg, i, l, tuned[i][l], bank) for l in range(cfg.num_layers)]
        counts = np.array([len(tuned[i][l]) for l in range(cfg.num_layers)], np.int32)
        ids = np.concatenate([tuned[i][l] for l in range(cfg.num_layers)]).astype(np.int32)
        pool.load_adapter(i, counts, ids, np.concatenate([e.w_gate for e in per_layer]),
                          np.concatenate([e.w_up for e in per_layer]), np.concatenate([e.w_down for e in per_layer]))
    return tuned, bases
