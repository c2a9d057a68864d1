"""ctypes binding of libgrowpage.so: the same entry points as `include/growpage.h`, with argument
marshalling only.  PyTorch supplies device memory and streams; every step of the path runs in the
library's CUDA kernels.  There is no fallback: a missing library raises at load time.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgrowpage.so")

GP_OK, GP_ERR_INVALID, GP_ERR_NO_SLOT, GP_ERR_NO_PAGES, GP_ERR_CUDA, GP_ERR_STATE = 0, -1, -2, -3, -4, -5
GP_ERR_TOO_LARGE = -6
GP_NOALLOC_MAX_ROWS = 2048
GP_ACT_NONE, GP_ACT_GROW, GP_ACT_COMPRESS, GP_ACT_COMPRESS_FALLBACK, GP_ACT_SHRINK = 0, 1, 2, 3, 4
GP_ACT_PENDING, GP_ACT_HELD = 5, 6
GP_ACT_STALLED, GP_ACT_SCRATCH, GP_ACT_INVALID = -1, -2, -3
GP_POLICY_DEMAND, GP_POLICY_INVERSE, GP_POLICY_RANDOM, GP_POLICY_SHRINK = 0, 1, 2, 3
GP_METRIC_TOP_P, GP_METRIC_ENTROPY = 0, 1
GP_N_KERNELS = 4
KERNEL_NAMES = ("plan", "attention", "boundary_or_select_decide", "compact_four_kernel_path")


class gp_config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("page_size", C.c_int32), ("max_requests", C.c_int32), ("max_pages_per_req", C.c_int32),
        ("recent_window", C.c_int32), ("k_loc", C.c_int32), ("host_staging", C.c_int32),
        ("policy", C.c_int32), ("policy_seed", C.c_int32), ("async_boundary", C.c_int32), ("demand_metric", C.c_int32),
        ("overlap_slots", C.c_int32), ("async_slots", C.c_int32),
        ("kv_shard_count", C.c_int32), ("reserved", C.c_int32),
        ("n_pages", C.c_int64), ("min_capacity", C.c_int64), ("max_batch_tokens", C.c_int64),
        ("max_boundary_tokens", C.c_int64),
        ("beta_s", C.c_double), ("beta_l", C.c_double), ("top_p", C.c_double), ("tau", C.c_double),
        ("rope_theta", C.c_double), ("p_compress", C.c_double), ("shrink_below", C.c_double),
    ]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Loads the library once.  Raises if it has not been built (`python -m paper_2609_03494_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_03494_b200.build`; "
                           "there is no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    L.gp_config_default.argtypes = [C.POINTER(gp_config)]
    L.gp_pool_bytes.argtypes = [C.POINTER(gp_config)]; L.gp_pool_bytes.restype = C.c_size_t
    L.gp_pool_create.argtypes = [C.POINTER(gp_config), vp, C.c_size_t, C.c_int, C.POINTER(vp)]
    L.gp_pool_destroy.argtypes = [vp]
    L.gp_request_add.argtypes = [vp, i32, i32, vp, vp, i32, i32, vp, C.POINTER(i32)]
    L.gp_decode_step.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.gp_decode_step_host.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.gp_decode_step_host_async.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.gp_decode_step_host_wait.argtypes = [vp]
    L.gp_decode_step_local.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.gp_shard_sums.argtypes = [vp, C.POINTER(C.c_void_p), C.POINTER(C.c_int64)]
    L.gp_decode_step_finish.argtypes = [vp, vp, i32, vp, vp]
    L.gp_release.argtypes = [vp, i32, vp]
    L.gp_strerror.argtypes = [C.c_int]; L.gp_strerror.restype = C.c_char_p
    L.gp_debug_request.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i64), vp]
    L.gp_debug_state.argtypes = [vp, vp, vp]
    L.gp_debug_retained.argtypes = [vp, i32, i32, i32, vp]
    L.gp_debug_kv.argtypes = [vp, i32, i32, i32, vp, vp]
    L.gp_debug_summaries.argtypes = [vp, i32, vp]
    L.gp_debug_boundary.argtypes = [vp, i32, vp, vp, C.POINTER(C.c_double)]
    L.gp_debug_pool.argtypes = [vp, C.POINTER(i64), vp, vp]
    L.gp_debug_entropy.argtypes = [vp, i32, vp, vp]
    L.gp_step_begin.argtypes = [vp, vp, i32, vp, vp]
    L.gp_attn_layer.argtypes = [vp, i32, vp, i32, vp, vp, vp, vp, vp]
    L.gp_step_end.argtypes = [vp, vp, i32, vp, vp]
    L.gp_attn_layer_qknorm.argtypes = [vp, i32, vp, i32, vp, vp, vp, vp, vp, C.c_double, vp, vp]
    L.gp_step_abort.argtypes = [vp]
    L.gp_pool_status.argtypes = [vp, C.POINTER(i32)]
    L.gp_async_join.argtypes = [vp, vp]
    L.gp_boundary_outcome.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i64)]
    L.gp_test_withhold.argtypes = [vp, i32, i32]
    L.gp_set_profiling.argtypes = [vp, i32]
    L.gp_set_early_plan.argtypes = [vp, i32]
    L.gp_get_kernel_times.argtypes = [vp, vp, vp]
    L.gp_launch_count.argtypes = [vp]; L.gp_launch_count.restype = i64
    L.gp_attention_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
    _lib = L
    return L


class GpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().gp_strerror(status).decode()} ({status})")


def _check(status: int, where: str) -> None:
    if status != GP_OK:
        raise GpError(status, where)


# ------------------------------------------------------------------------------- same names as the C ABI
def gp_config_default() -> gp_config:
    cfg = gp_config()
    _check(lib().gp_config_default(C.byref(cfg)), "gp_config_default")
    return cfg


def gp_pool_bytes(cfg: gp_config) -> int:
    return int(lib().gp_pool_bytes(C.byref(cfg)))


def gp_pool_create(cfg: gp_config, dev_blob_ptr: int, nbytes: int, device: int) -> int:
    handle = C.c_void_p()
    _check(lib().gp_pool_create(C.byref(cfg), C.c_void_p(dev_blob_ptr), nbytes, device, C.byref(handle)),
           "gp_pool_create")
    return handle.value


def gp_pool_destroy(pool: int) -> None:
    _check(lib().gp_pool_destroy(C.c_void_p(pool)), "gp_pool_destroy")


def gp_request_add(pool: int, share_from: int, n_shared_pages: int, k_tail_ptr: int, v_tail_ptr: int, n_tail: int,
                   initial_pages: int, stream: int) -> Tuple[int, int]:
    """Returns (status, request id); the status is returned, not raised, so that a scheduler can
    react to GP_ERR_NO_PAGES / GP_ERR_NO_SLOT."""
    rid = C.c_int32(-1)
    st = lib().gp_request_add(C.c_void_p(pool), share_from, n_shared_pages, C.c_void_p(k_tail_ptr),
                              C.c_void_p(v_tail_ptr), n_tail, initial_pages, C.c_void_p(stream), C.byref(rid))
    return int(st), int(rid.value)


def gp_decode_step(pool: int, dev_req_ids_ptr: int, n_req: int, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int,
                   dev_actions_ptr: int, stream: int) -> None:
    _check(lib().gp_decode_step(C.c_void_p(pool), C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(q_ptr),
                                C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(out_ptr),
                                C.c_void_p(dev_actions_ptr), C.c_void_p(stream)), "gp_decode_step")


def gp_decode_step_host(pool: int, host_req_ids_ptr: int, n_req: int, q_ptr: int, k_ptr: int, v_ptr: int,
                        out_ptr: int, actions_ptr: int, stream: int) -> None:
    _check(lib().gp_decode_step_host(C.c_void_p(pool), C.c_void_p(host_req_ids_ptr), n_req, C.c_void_p(q_ptr),
                                     C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(out_ptr),
                                     C.c_void_p(actions_ptr), C.c_void_p(stream)), "gp_decode_step_host")


def gp_decode_step_host_async(pool: int, host_req_ids_ptr: int, n_req: int, q_ptr: int, k_ptr: int, v_ptr: int,
                              out_ptr: int, actions_ptr: int, stream: int) -> None:
    _check(lib().gp_decode_step_host_async(C.c_void_p(pool), C.c_void_p(host_req_ids_ptr), n_req, C.c_void_p(q_ptr),
                                           C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(out_ptr),
                                           C.c_void_p(actions_ptr), C.c_void_p(stream)), "gp_decode_step_host_async")


def gp_step_begin(pool: int, dev_req_ids_ptr: int, n_req: int, dev_actions_ptr: int, stream: int) -> None:
    _check(lib().gp_step_begin(C.c_void_p(pool), C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(dev_actions_ptr),
                               C.c_void_p(stream)), "gp_step_begin")


def gp_attn_layer(pool: int, layer: int, dev_req_ids_ptr: int, n_req: int, q_ptr: int, k_ptr: int, v_ptr: int,
                  out_ptr: int, stream: int) -> None:
    _check(lib().gp_attn_layer(C.c_void_p(pool), layer, C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(q_ptr),
                               C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(out_ptr), C.c_void_p(stream)),
           "gp_attn_layer")


def gp_attn_layer_qknorm(pool: int, layer: int, dev_req_ids_ptr: int, n_req: int, q_raw_ptr: int, k_raw_ptr: int, v_ptr: int,
                         q_weight_ptr: int, k_weight_ptr: int, eps: float, out_ptr: int, stream: int) -> None:
    _check(lib().gp_attn_layer_qknorm(C.c_void_p(pool), layer, C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(q_raw_ptr),
                                      C.c_void_p(k_raw_ptr), C.c_void_p(v_ptr), C.c_void_p(q_weight_ptr),
                                      C.c_void_p(k_weight_ptr), eps, C.c_void_p(out_ptr), C.c_void_p(stream)),
           "gp_attn_layer_qknorm")


def gp_step_end(pool: int, dev_req_ids_ptr: int, n_req: int, dev_actions_ptr: int, stream: int) -> None:
    _check(lib().gp_step_end(C.c_void_p(pool), C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(dev_actions_ptr),
                             C.c_void_p(stream)), "gp_step_end")


def gp_step_abort(pool: int) -> None:
    _check(lib().gp_step_abort(C.c_void_p(pool)), "gp_step_abort")


def gp_decode_step_host_wait(pool: int) -> None:
    _check(lib().gp_decode_step_host_wait(C.c_void_p(pool)), "gp_decode_step_host_wait")


def gp_decode_step_local(pool: int, dev_req_ids_ptr: int, n_req: int, q_ptr: int, k_ptr: int, v_ptr: int,
                         out_ptr: int, dev_actions_ptr: int, stream: int) -> None:
    _check(lib().gp_decode_step_local(C.c_void_p(pool), C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(q_ptr),
                                      C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(out_ptr),
                                      C.c_void_p(dev_actions_ptr), C.c_void_p(stream)), "gp_decode_step_local")


def gp_shard_sums(pool: int) -> Tuple[int, int]:
    """Device address and length (int32 elements) of the array to be summed over the KV-head shards."""
    ptr = C.c_void_p(0)
    n = C.c_int64(0)
    _check(lib().gp_shard_sums(C.c_void_p(pool), C.byref(ptr), C.byref(n)), "gp_shard_sums")
    return int(ptr.value), int(n.value)


def gp_decode_step_finish(pool: int, dev_req_ids_ptr: int, n_req: int, dev_actions_ptr: int, stream: int) -> None:
    _check(lib().gp_decode_step_finish(C.c_void_p(pool), C.c_void_p(dev_req_ids_ptr), n_req, C.c_void_p(dev_actions_ptr),
                                       C.c_void_p(stream)), "gp_decode_step_finish")


def gp_pool_status(pool: int) -> Tuple[int, int]:
    """Returns (status, error bits) of the kernels' error word; the status is returned, not raised."""
    bits = C.c_int32(0)
    st = lib().gp_pool_status(C.c_void_p(pool), C.byref(bits))
    return int(st), int(bits.value)


def gp_async_join(pool: int, stream: int) -> None:
    _check(lib().gp_async_join(C.c_void_p(pool), C.c_void_p(stream)), "gp_async_join")


def gp_boundary_outcome(pool: int, req: int) -> Tuple[int, int]:
    """(action, step) of the request's most recent capacity boundary."""
    act, step = C.c_int32(0), C.c_int64(-1)
    _check(lib().gp_boundary_outcome(C.c_void_p(pool), req, C.byref(act), C.byref(step)), "gp_boundary_outcome")
    return int(act.value), int(step.value)


def gp_release(pool: int, req: int, stream: int) -> None:
    _check(lib().gp_release(C.c_void_p(pool), req, C.c_void_p(stream)), "gp_release")


def gp_strerror(status: int) -> str:
    return lib().gp_strerror(status).decode()


def gp_debug_request(pool: int, req: int, cap: int):
    P, n, pos = C.c_int32(), C.c_int32(), C.c_int64()
    table = np.zeros(cap, dtype=np.int32)
    _check(lib().gp_debug_request(C.c_void_p(pool), req, C.byref(P), C.byref(n), C.byref(pos),
                                  table.ctypes.data_as(C.c_void_p)), "gp_debug_request")
    return int(P.value), int(n.value), int(pos.value), table[:P.value].tolist()


def gp_debug_state(pool: int, max_requests: int) -> Tuple[np.ndarray, np.ndarray]:
    P = np.zeros(max_requests, dtype=np.int32)
    n = np.zeros(max_requests, dtype=np.int32)
    _check(lib().gp_debug_state(C.c_void_p(pool), P.ctypes.data_as(C.c_void_p), n.ctypes.data_as(C.c_void_p)),
           "gp_debug_state")
    return P, n


def gp_debug_retained(pool: int, req: int, layer: int, kv_head: int, n: int) -> np.ndarray:
    out = np.zeros(max(n, 1), dtype=np.int32)
    _check(lib().gp_debug_retained(C.c_void_p(pool), req, layer, kv_head, out.ctypes.data_as(C.c_void_p)),
           "gp_debug_retained")
    return out[:n]


def gp_debug_kv(pool: int, req: int, layer: int, kv_head: int, n: int, d: int):
    k = np.zeros((max(n, 1), d), dtype=np.uint16)
    v = np.zeros((max(n, 1), d), dtype=np.uint16)
    _check(lib().gp_debug_kv(C.c_void_p(pool), req, layer, kv_head, k.ctypes.data_as(C.c_void_p),
                             v.ctypes.data_as(C.c_void_p)), "gp_debug_kv")
    return k[:n], v[:n]


def gp_debug_summaries(pool: int, req: int, L: int, Hq: int, d: int) -> np.ndarray:
    out = np.zeros((L, 2, Hq, d), dtype=np.float64)
    _check(lib().gp_debug_summaries(C.c_void_p(pool), req, out.ctypes.data_as(C.c_void_p)), "gp_debug_summaries")
    return out


def gp_debug_boundary(pool: int, req: int, L: int, Hkv: int):
    ks = np.zeros((L, Hkv), dtype=np.int32)
    kl = np.zeros((L, Hkv), dtype=np.int32)
    delta = C.c_double()
    _check(lib().gp_debug_boundary(C.c_void_p(pool), req, ks.ctypes.data_as(C.c_void_p),
                                   kl.ctypes.data_as(C.c_void_p), C.byref(delta)), "gp_debug_boundary")
    return ks, kl, float(delta.value)


def gp_debug_entropy(pool: int, req: int, L: int, Hkv: int):
    hs = np.zeros((L, Hkv), dtype=np.float64)
    hl = np.zeros((L, Hkv), dtype=np.float64)
    _check(lib().gp_debug_entropy(C.c_void_p(pool), req, hs.ctypes.data_as(C.c_void_p), hl.ctypes.data_as(C.c_void_p)),
           "gp_debug_entropy")
    return hs, hl


def gp_debug_pool(pool: int, n_pages: int = 0):
    n_free = C.c_int64()
    counters = np.zeros(12, dtype=np.int64)
    ref = np.zeros(max(n_pages, 1), dtype=np.int32)
    _check(lib().gp_debug_pool(C.c_void_p(pool), C.byref(n_free), ref.ctypes.data_as(C.c_void_p) if n_pages else None,
                               counters.ctypes.data_as(C.c_void_p)), "gp_debug_pool")
    return int(n_free.value), ref[:n_pages], counters


def gp_test_withhold(pool: int, what: int, spin_limit: int) -> None:
    _check(lib().gp_test_withhold(C.c_void_p(pool), what, spin_limit), "gp_test_withhold")


def gp_set_early_plan(pool: int, enable: bool) -> None:
    _check(lib().gp_set_early_plan(C.c_void_p(pool), 1 if enable else 0), "gp_set_early_plan")


def gp_set_profiling(pool: int, enable: bool) -> None:
    _check(lib().gp_set_profiling(C.c_void_p(pool), 1 if enable else 0), "gp_set_profiling")


def gp_get_kernel_times(pool: int):
    ms = np.zeros(GP_N_KERNELS, dtype=np.float32)
    n = np.zeros(GP_N_KERNELS, dtype=np.int64)
    _check(lib().gp_get_kernel_times(C.c_void_p(pool), ms.ctypes.data_as(C.c_void_p), n.ctypes.data_as(C.c_void_p)),
           "gp_get_kernel_times")
    return ms, n


def gp_launch_count(pool: int) -> int:
    return int(lib().gp_launch_count(C.c_void_p(pool)))


def gp_attention_noalloc(q_ptr: int, k_ptr: int, v_ptr: int, lens_ptr: int, n_req: int, n_q_heads: int,
                         n_kv_heads: int, head_dim: int, max_len: int, out_ptr: int, stream: int) -> None:
    """Decode attention over plain K/V for callers that may not allocate: the library brings its own fixed
    scratch.  All pointers are device addresses the caller owns; raises GpError (GP_ERR_TOO_LARGE when
    n_req * n_q_heads exceeds GP_NOALLOC_MAX_ROWS).  Do not overlap two calls on the GPU."""
    _check(lib().gp_attention_noalloc(C.c_void_p(q_ptr), C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(lens_ptr),
                                      n_req, n_q_heads, n_kv_heads, head_dim, max_len, C.c_void_p(out_ptr),
                                      C.c_void_p(stream)), "gp_attention_noalloc")


# ------------------------------------------------------------------------------- convenience holder
class Pool:
    """Owns the torch blob and the handle of one pool, and marshals torch tensors into the calls above."""

    def __init__(self, cfg: gp_config, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required; there is no CPU fallback")
        self.torch = torch
        self.cfg = cfg
        self.device = device
        nbytes = gp_pool_bytes(cfg)
        if nbytes == 0:
            raise GpError(GP_ERR_INVALID, "gp_pool_bytes")
        self.nbytes = nbytes
        self.blob = torch.empty(nbytes + 256, dtype=torch.uint8, device=f"cuda:{device}")
        base = (self.blob.data_ptr() + 255) & ~255
        self.handle = gp_pool_create(cfg, base, nbytes, device)

    def stream(self) -> int:
        return int(self.torch.cuda.current_stream(self.device).cuda_stream)

    def request_add(self, share_from: int, n_shared_pages: int, k_tail, v_tail, n_tail: int, initial_pages: int):
        """k_tail / v_tail: uint16 numpy [L][n_tail][H_kv][d] (bf16 bits), torch device tensors, or None."""
        torch = self.torch
        kp = vp = 0
        keep = []
        if n_tail:
            for name, x in (("k", k_tail), ("v", v_tail)):
                if isinstance(x, np.ndarray):
                    x = torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(f"cuda:{self.device}")
                keep.append(x.contiguous())
            kp, vp = keep[0].data_ptr(), keep[1].data_ptr()
        return gp_request_add(self.handle, share_from, n_shared_pages, kp, vp, n_tail, initial_pages, self.stream())

    def decode_step(self, req_ids, q, k, v, out, actions) -> None:
        """All arguments are torch CUDA tensors: req_ids int32 [B], q/k/v bf16 (or int16 bit views), out fp32,
        actions int32 [B]."""
        gp_decode_step(self.handle, req_ids.data_ptr(), int(req_ids.numel()), q.data_ptr(), k.data_ptr(),
                       v.data_ptr(), out.data_ptr(), actions.data_ptr(), self.stream())

    def decode_step_layers(self, req_ids, q, k, v, out, actions) -> None:
        """The same step through the per-layer entry points: q, k, v, out as for decode_step ([L][...]); every
        layer's slice is passed to gp_attn_layer on its own."""
        n = int(req_ids.numel())
        gp_step_begin(self.handle, req_ids.data_ptr(), n, actions.data_ptr(), self.stream())
        for layer in range(q.shape[0]):
            gp_attn_layer(self.handle, layer, req_ids.data_ptr(), n, q[layer].data_ptr(), k[layer].data_ptr(),
                          v[layer].data_ptr(), out[layer].data_ptr(), self.stream())
        gp_step_end(self.handle, req_ids.data_ptr(), n, actions.data_ptr(), self.stream())

    def decode_step_host(self, req_ids, q, k, v, out, actions) -> None:
        """All arguments are host tensors (pinned recommended)."""
        gp_decode_step_host(self.handle, req_ids.data_ptr(), int(req_ids.numel()), q.data_ptr(), k.data_ptr(),
                            v.data_ptr(), out.data_ptr(), actions.data_ptr(), self.stream())

    def decode_step_host_async(self, req_ids, q, k, v, out, actions) -> None:
        """As decode_step_host, without the synchronisation at the end: results are there once host_wait has returned
        for the call."""
        gp_decode_step_host_async(self.handle, req_ids.data_ptr(), int(req_ids.numel()), q.data_ptr(), k.data_ptr(),
                                  v.data_ptr(), out.data_ptr(), actions.data_ptr(), self.stream())

    def host_wait(self) -> None:
        gp_decode_step_host_wait(self.handle)

    def release(self, req: int) -> None:
        gp_release(self.handle, req, self.stream())

    def close(self) -> None:
        if self.handle:
            gp_pool_destroy(self.handle)
            self.handle = 0
            self.blob = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_config(n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_pages: int, max_pages_per_req: int,
                max_requests: int = 512, k_loc: int = 4, host_staging: bool = False, max_batch_tokens: int = 0,
                beta_s: float = 0.9, beta_l: float = 0.999, top_p: float = 0.99, tau: float = 0.0,
                rope_theta: float = 0.0, policy: int = 0, policy_seed: int = 0, p_compress: float = 0.7,
                shrink_below: float = -0.005, min_capacity: int = 1024, async_boundary: bool = False,
                async_slots: int = 0, max_boundary_tokens: int = 0, demand_metric: int = 0, page_size: int = 16,
                overlap_slots: int = 0, kv_shard_count: int = 1) -> gp_config:
    cfg = gp_config_default()
    cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
    cfg.n_pages, cfg.max_pages_per_req, cfg.max_requests = n_pages, max_pages_per_req, max_requests
    cfg.k_loc, cfg.host_staging, cfg.max_batch_tokens = k_loc, 1 if host_staging else 0, max_batch_tokens
    cfg.beta_s, cfg.beta_l, cfg.top_p, cfg.tau, cfg.rope_theta = beta_s, beta_l, top_p, tau, rope_theta
    cfg.policy, cfg.policy_seed, cfg.p_compress = policy, policy_seed, p_compress
    cfg.shrink_below, cfg.min_capacity = shrink_below, min_capacity
    cfg.async_boundary, cfg.async_slots, cfg.max_boundary_tokens = 1 if async_boundary else 0, async_slots, max_boundary_tokens
    cfg.overlap_slots = overlap_slots
    cfg.kv_shard_count = kv_shard_count
    cfg.demand_metric = demand_metric
    cfg.page_size = page_size
    return cfg
