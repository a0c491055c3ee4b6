"""ctypes binding of include/mira.h (argument marshalling only) and the `Mira` helper class."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmira.so")

MIRA_OK, MIRA_ERR_INVALID_ARG, MIRA_ERR_SHAPE, MIRA_ERR_ALIGN, MIRA_ERR_EXPERT_MISS = 0, 1, 2, 3, 4
MIRA_ERR_NO_PREDICTOR, MIRA_ERR_WORKSPACE, MIRA_ERR_CUDA, MIRA_ERR_UNSUPPORTED, MIRA_ERR_TIMEOUT = 5, 6, 7, 8, 9


class mira_config(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("ffn", C.c_int32), ("n_experts", C.c_int32),
                ("n_shared", C.c_int32), ("n_layers", C.c_int32), ("max_tokens", C.c_int32),
                ("max_top_k", C.c_int32), ("act_on_w1", C.c_int32), ("out_dtype", C.c_int32),
                ("eps", C.c_float), ("format", C.c_int32)]


class mira_mixture_head(C.Structure):
    _fields_ = [("wa_h", C.c_void_p), ("wa_l", C.c_void_p), ("b_a", C.c_void_p), ("wh_c", C.c_void_p),
                ("wh_t", C.c_void_p), ("b_h", C.c_void_p), ("g_h", C.c_void_p), ("g_l", C.c_void_p),
                ("g_c", C.c_void_p), ("b_g", C.c_float)]


class mira_stack_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_hot", C.c_int32), ("n_stage", C.c_int32), ("k_pred", C.c_int32),
                ("rebalance_every", C.c_int32), ("max_swaps", C.c_int32), ("miss_weight", C.c_float),
                ("margin", C.c_float)]


class mira_route_out(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("w", C.c_void_p), ("count", C.c_void_p), ("offset", C.c_void_p),
                ("perm", C.c_void_p), ("logits", C.c_void_p)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_38090_b200.build` "
            "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    cfgp = C.POINTER(mira_config)
    ip = C.POINTER(C.c_int32)
    sig = {
        "mira_expert_bytes": (sz, [i32, i32]),
        "mira_expert_bytes_format": (sz, [i32, i32, i32]),
        "mira_workspace_bytes": (sz, [cfgp]),
        "mira_create": (C.c_int, [cfgp, vp, sz, C.POINTER(vp)]),
        "mira_destroy": (None, [vp]),
        "mira_quantize_experts": (C.c_int, [vp, vp, vp, vp, i32, i32, vp, vp]),
        "mira_unpack_expert": (C.c_int, [vp, vp, vp, vp, vp, vp, vp, vp, vp]),
        "mira_stage_expert": (C.c_int, [vp, vp, vp, vp, vp]),
        "mira_predict": (C.c_int, [vp, i32, vp, i32, vp, vp, vp, vp, vp, i32, vp]),
        "mira_predict_noalloc": (C.c_int, [vp, i32, i32, vp, vp, i32, vp, vp, i32, vp]),
        "mira_predict_mixture": (C.c_int, [vp, i32, vp, i32, vp, vp, i32, C.POINTER(mira_mixture_head), vp, vp, vp, vp,
                                           i32, vp]),
        "mira_moe_layer": (C.c_int, [vp, vp, i32, vp, vp, vp, vp, i32, vp, C.POINTER(mira_route_out), vp]),
        "mira_route": (C.c_int, [vp, vp, i32, vp, vp, i32, C.POINTER(mira_route_out), vp]),
        "mira_moe_experts": (C.c_int, [vp, vp, i32, vp, vp, C.POINTER(C.c_uint32), i32, vp, vp]),
        "mira_poll_status": (C.c_int, [vp, C.POINTER(C.c_uint32), vp]),
        "mira_kernel_launches": (C.c_int64, [vp]),
        "mira_set_option": (C.c_int, [vp, i32, i32]),
        "mira_profile": (C.c_int, [vp, i32]),
        "mira_profile_read": (C.c_int, [vp, C.POINTER(C.c_float), C.POINTER(C.c_int64)]),
        "mira_status_string": (C.c_char_p, [C.c_int]),
        "mira_cache_budget": (C.c_int, [C.c_int64, C.c_int64, C.c_int64, i32, i32, i32, i32, ip, ip, ip]),
        "mira_cache_create": (C.c_int, [i32, i32, ip, i32, i32, C.POINTER(vp)]),
        "mira_cache_destroy": (None, [vp]),
        "mira_cache_slot_map": (C.c_int, [vp, ip]),
        "mira_cache_prefetch": (i32, [vp, ip, i32, ip, ip]),
        "mira_cache_plan": (i32, [vp, ip, ip, ip, ip, i32]),
        "mira_cache_layer_done": (None, [vp, i32]),
        "mira_cache_rebalance": (i32, [vp, i32, C.c_float, C.c_float, ip, ip, ip]),
        "mira_cache_stats": (None, [vp, C.POINTER(C.c_int64)]),
        "mira_cache_stats_reset": (None, [vp]),
        "mira_stack_scratch_bytes": (sz, [vp, C.POINTER(mira_stack_config)]),
        "mira_stack_create": (C.c_int, [vp, C.POINTER(mira_stack_config), C.POINTER(vp), C.POINTER(vp), ip, vp, sz, vp, vp,
                                        C.POINTER(vp)]),
        "mira_stack_destroy": (None, [vp]),
        "mira_stack_layer_step": (C.c_int, [vp, i32, vp, i32, vp, vp, i32, vp, vp, vp, vp]),
        "mira_stack_stats": (C.c_int, [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
        "mira_stack_stats_reset": (None, [vp]),
        "mira_stack_coverage": (C.c_int, [vp, C.POINTER(C.c_double), ip]),
        "mira_stack_cache": (vp, [vp, i32]),
        "mira_residual_rmsnorm": (C.c_int, [vp, vp, i32, i32, C.c_float, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()

# The C entry points under their own names.
mira_expert_bytes = lib.mira_expert_bytes
mira_expert_bytes_format = lib.mira_expert_bytes_format
MIRA_FORMAT_SHARED, MIRA_FORMAT_PER_MATRIX = 0, 1
mira_workspace_bytes = lib.mira_workspace_bytes
mira_create = lib.mira_create
mira_destroy = lib.mira_destroy
mira_quantize_experts = lib.mira_quantize_experts
mira_unpack_expert = lib.mira_unpack_expert
mira_stage_expert = lib.mira_stage_expert
mira_predict = lib.mira_predict
mira_predict_noalloc = lib.mira_predict_noalloc
mira_predict_mixture = lib.mira_predict_mixture
mira_moe_layer = lib.mira_moe_layer
mira_route = lib.mira_route
mira_moe_experts = lib.mira_moe_experts
mira_poll_status = lib.mira_poll_status
mira_kernel_launches = lib.mira_kernel_launches
mira_profile = lib.mira_profile
mira_set_option = lib.mira_set_option
MIRA_OPT_FORCE_DECODE_PATH = 1
MIRA_OPT_TENSOR_LAYOUT = 2
MIRA_OPT_UP_CONVERSION = 3
MIRA_OPT_TEST_WAIT_TIMEOUT = 4
MIRA_OPT_HYBRID_MIN_UP = 5
MIRA_OPT_HYBRID_MIN_DOWN = 6
MIRA_OPT_DOWN_SLICES = 7
mira_profile_read = lib.mira_profile_read
KERNEL_CLASSES = ("route", "group", "schedule", "up_gate", "down", "combine", "scores", "pool", "quantize", "unpack")
mira_status_string = lib.mira_status_string
mira_cache_budget = lib.mira_cache_budget
mira_cache_create = lib.mira_cache_create
mira_cache_destroy = lib.mira_cache_destroy
mira_cache_slot_map = lib.mira_cache_slot_map
mira_cache_prefetch = lib.mira_cache_prefetch
mira_cache_plan = lib.mira_cache_plan
mira_cache_layer_done = lib.mira_cache_layer_done
mira_cache_rebalance = lib.mira_cache_rebalance
mira_cache_stats = lib.mira_cache_stats
mira_cache_stats_reset = lib.mira_cache_stats_reset
mira_stack_scratch_bytes = lib.mira_stack_scratch_bytes
mira_stack_create = lib.mira_stack_create
mira_stack_destroy = lib.mira_stack_destroy
mira_stack_layer_step = lib.mira_stack_layer_step
mira_stack_stats = lib.mira_stack_stats
mira_stack_stats_reset = lib.mira_stack_stats_reset
mira_stack_coverage = lib.mira_stack_coverage
mira_stack_cache = lib.mira_stack_cache
mira_residual_rmsnorm = lib.mira_residual_rmsnorm


class MiraError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {mira_status_string(code).decode()} (status {code})")


def _check(code: int, where: str) -> None:
    if code != MIRA_OK:
        raise MiraError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


class Mira:
    """One library context plus its workspace tensor. Methods take CUDA tensors and pass raw pointers."""

    def __init__(self, hidden: int, ffn: int, n_experts: int, n_shared: int = 0, n_layers: int = 0,
                 max_tokens: int = 64, max_top_k: int = 2, act_on_w1: bool = False, out_fp32: bool = False,
                 eps: float = 1e-8, device: str | torch.device = "cuda:0", fmt: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("Mira needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.cfg = mira_config(hidden, ffn, n_experts, n_shared, n_layers, max_tokens, max_top_k,
                               int(act_on_w1), int(out_fp32), eps, fmt)
        nbytes = mira_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise MiraError(MIRA_ERR_SHAPE, "mira_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self._ctx = C.c_void_p()
        _check(mira_create(C.byref(self.cfg), C.c_void_p(base), nbytes, C.byref(self._ctx)), "mira_create")
        self.C, self.R, self.E, self.ns = hidden, ffn, n_experts, n_shared
        self.out_dtype = torch.float32 if out_fp32 else torch.bfloat16
        self.expert_bytes = mira_expert_bytes_format(ffn, hidden, fmt)

    def close(self):
        if getattr(self, "_ctx", None) and mira_destroy is not None:      # module globals are gone at interpreter exit
            mira_destroy(self._ctx)
            self._ctx = None

    __del__ = close

    # S0 ------------------------------------------------------------------------------------
    def quantize_experts(self, w1, w2, w3, out=None, stream=None):
        """w1, w3 [n,R,C], w2 [n,C,R] (fp32 or bf16, CUDA) -> blobs [n, expert_bytes] uint8."""
        n = w1.shape[0]
        assert w1.shape == (n, self.R, self.C) and w3.shape == w1.shape and w2.shape == (n, self.C, self.R)
        assert w1.dtype == w2.dtype == w3.dtype and w1.dtype in (torch.float32, torch.bfloat16)
        w1, w2, w3 = w1.contiguous(), w2.contiguous(), w3.contiguous()
        if out is None:
            out = torch.empty((n, self.expert_bytes), dtype=torch.uint8, device=self.device)
        _check(mira_quantize_experts(self._ctx, _ptr(w1), _ptr(w2), _ptr(w3), 0 if w1.dtype == torch.float32 else 1,
                                     n, _ptr(out), _stream(stream)), "mira_quantize_experts")
        return out

    def unpack_expert(self, blob, codes=True, weights=True, stream=None):
        R, Cc = self.R, self.C
        o = {}
        if codes:
            o.update(q1=torch.empty((R, Cc), dtype=torch.int8, device=self.device),
                     q2=torch.empty((Cc, R), dtype=torch.int8, device=self.device),
                     q3=torch.empty((R, Cc), dtype=torch.int8, device=self.device))
        if weights:
            o.update(w1=torch.empty((R, Cc), dtype=torch.float32, device=self.device),
                     w2=torch.empty((Cc, R), dtype=torch.float32, device=self.device),
                     w3=torch.empty((R, Cc), dtype=torch.float32, device=self.device))
        _check(mira_unpack_expert(self._ctx, _ptr(blob), _ptr(o.get("q1")), _ptr(o.get("q2")), _ptr(o.get("q3")),
                                  _ptr(o.get("w1")), _ptr(o.get("w2")), _ptr(o.get("w3")), _stream(stream)),
               "mira_unpack_expert")
        return o

    # S8 ------------------------------------------------------------------------------------
    def stage_expert(self, pinned_blob, dev_slot, side_stream, ready_event=None):
        assert pinned_blob.is_pinned() and pinned_blob.numel() >= self.expert_bytes
        if ready_event is not None and not ready_event.cuda_event:
            # torch creates the CUDA event on its first record(); a handle of 0 would make the C call skip the
            # record. This extra record (before the copy) is overwritten by the one after the copy.
            ready_event.record(side_stream)
        ev = None if ready_event is None else C.c_void_p(ready_event.cuda_event)
        assert ev is None or ev.value, "ready_event has no CUDA event handle"
        _check(mira_stage_expert(self._ctx, C.c_void_p(pinned_blob.data_ptr()), _ptr(dev_slot),
                                 C.c_void_p(side_stream.cuda_stream), ev), "mira_stage_expert")

    # S7 ------------------------------------------------------------------------------------
    def predict(self, layer, hidden, pred_w, pred_b=None, k_pred=2, token_scores=False, stream=None, reuse=False):
        """reuse=True returns the same output tensors on every call with the same (T, k_pred, token_scores)."""
        T = hidden.shape[0]
        key = ("predict", T, k_pred, bool(token_scores))
        cache = self.__dict__.setdefault("_out_cache", {})
        if reuse and key in cache:
            pooled, ts, ids = cache[key]
        else:
            pooled = torch.empty(self.E, dtype=torch.float32, device=self.device)
            ts = torch.empty((T, self.E), dtype=torch.float32, device=self.device) if token_scores else None
            ids = torch.empty(max(k_pred, 1), dtype=torch.int32, device=self.device) if k_pred > 0 else None
            if reuse:
                cache[key] = (pooled, ts, ids)
        _check(mira_predict(self._ctx, layer, _ptr(hidden), T, _ptr(pred_w), _ptr(pred_b), _ptr(pooled), _ptr(ts),
                            _ptr(ids), k_pred, _stream(stream)), "mira_predict")
        return pooled, ts, (ids[:k_pred] if ids is not None else None)

    def predict_mixture(self, layer, hidden, router_logits, count, k_top, head: dict, k_pred=2, stream=None):
        """MixtureHead on the by-products of mira_route. head: CUDA tensors wa_h, wa_l, wh_c, wh_t (bf16 matrices),
        g_h, g_l, g_c (bf16 vectors), b_a, b_h (fp32 vectors) and the float b_g. Returns (scores, probs, alpha, ids)."""
        T = hidden.shape[0]
        hs = mira_mixture_head(*(head[n].data_ptr() for n in ("wa_h", "wa_l", "b_a", "wh_c", "wh_t", "b_h", "g_h", "g_l", "g_c")),
                               float(head["b_g"]))
        scores = torch.empty(self.E, dtype=torch.float32, device=self.device)
        probs = torch.empty(self.E, dtype=torch.float32, device=self.device)
        alpha = torch.empty(1, dtype=torch.float32, device=self.device)
        ids = torch.empty(max(k_pred, 1), dtype=torch.int32, device=self.device)
        _check(mira_predict_mixture(self._ctx, layer, _ptr(hidden), T, _ptr(router_logits), _ptr(count), k_top, C.byref(hs),
                                    _ptr(scores), _ptr(probs), _ptr(alpha), _ptr(ids), k_pred, _stream(stream)),
               "mira_predict_mixture")
        return scores, probs, alpha, ids[:k_pred]

    # S1-S6 ---------------------------------------------------------------------------------
    def _route_buffers(self, T, k, logits=True):
        dev, kk, Et = self.device, k + self.ns, self.E + self.ns
        b = dict(idx=torch.empty((T, k), dtype=torch.int32, device=dev),
                 w=torch.empty((T, k), dtype=torch.float32, device=dev),
                 count=torch.empty(Et, dtype=torch.int32, device=dev),
                 offset=torch.empty(Et + 1, dtype=torch.int32, device=dev),
                 perm=torch.empty((T, kk), dtype=torch.int32, device=dev))
        if logits:
            b["logits"] = torch.empty((T, self.E), dtype=torch.float32, device=dev)
        st = mira_route_out(*(b[n].data_ptr() if n in b else None
                              for n in ("idx", "w", "count", "offset", "perm", "logits")))
        return b, st

    def moe_layer(self, hidden, router_w, router_bias, expert_slots, slot_map, k, out=None, debug=False,
                  stream=None):
        """hidden [T,C] bf16; expert_slots: int64 CUDA tensor of slot base addresses; slot_map int32 [E+ns]."""
        T = hidden.shape[0]
        if out is None:
            out = torch.empty((T, self.C), dtype=self.out_dtype, device=self.device)
        bufs, st = self._route_buffers(T, k) if debug else (None, None)
        _check(mira_moe_layer(self._ctx, _ptr(hidden), T, _ptr(router_w), _ptr(router_bias), _ptr(expert_slots),
                              _ptr(slot_map), k, _ptr(out), C.byref(st) if st is not None else None,
                              _stream(stream)), "mira_moe_layer")
        return (out, bufs) if debug else out

    def route(self, hidden, router_w, router_bias, k, stream=None, reuse=False):
        """S1-S3. reuse=True returns the same output tensors on every call with the same (T, k): for callers
        that consume the result before routing again (no allocation per call)."""
        T = hidden.shape[0]
        if reuse:
            cache = self.__dict__.setdefault("_route_cache", {})
            if (T, k) not in cache:
                cache[(T, k)] = self._route_buffers(T, k)
            bufs, st = cache[(T, k)]
        else:
            bufs, st = self._route_buffers(T, k)
        _check(mira_route(self._ctx, _ptr(hidden), T, _ptr(router_w), _ptr(router_bias), k, C.byref(st),
                          _stream(stream)), "mira_route")
        return bufs

    def moe_experts(self, hidden, expert_slots, slot_map, expert_ids=None, final_wave=True, out=None, stream=None):
        T = hidden.shape[0]
        mask = None
        if expert_ids is not None:
            words = (self.E + self.ns + 31) // 32
            mask = (C.c_uint32 * words)()
            for e in expert_ids:
                mask[e >> 5] |= 1 << (e & 31)
        if final_wave and out is None:
            out = torch.empty((T, self.C), dtype=self.out_dtype, device=self.device)
        _check(mira_moe_experts(self._ctx, _ptr(hidden), T, _ptr(expert_slots), _ptr(slot_map), mask,
                                int(final_wave), _ptr(out), _stream(stream)), "mira_moe_experts")
        return out

    def poll_status(self, stream=None):
        """Synchronises; returns (status code, list of missing expert ids)."""
        words = (self.E + self.ns + 31) // 32
        mask = (C.c_uint32 * words)()
        code = mira_poll_status(self._ctx, mask, _stream(stream))
        missing = [e for e in range(self.E + self.ns) if (mask[e >> 5] >> (e & 31)) & 1] if code in (MIRA_ERR_EXPERT_MISS, MIRA_ERR_TIMEOUT) else []
        return code, missing

    def force_decode_path(self, on: bool) -> None:
        _check(mira_set_option(self._ctx, MIRA_OPT_FORCE_DECODE_PATH, int(on)), "mira_set_option")

    def tensor_layout(self, layout: int) -> None:
        """0: chosen per step (default); 1, 2, 3: force the narrow, wide or big tile layout of the tensor-core kernels;
        4, 5: the two-SM (cta_group::2) kernel with 192-token tiles x 4 stages or 128-token tiles x 8 stages."""
        _check(mira_set_option(self._ctx, MIRA_OPT_TENSOR_LAYOUT, int(layout)), "mira_set_option")

    def up_conversion(self, mode: int) -> None:
        """tcgen05 up/gate kernel: 0, 1: exact code conversion (default); 2: offset subnormals (faster, input-dependent accuracy)."""
        _check(mira_set_option(self._ctx, MIRA_OPT_UP_CONVERSION, int(mode)), "mira_set_option")

    def hybrid_min(self, up: int = -1, down: int = -1) -> None:
        """Pair count from which an expert goes to the tcgen05 kernel of the up/gate and of the down projection
        (-1: the library's rule; 0: all; 2**31 - 1: none). Set before the step's routing call."""
        _check(mira_set_option(self._ctx, MIRA_OPT_HYBRID_MIN_UP, int(up)), "mira_set_option")
        _check(mira_set_option(self._ctx, MIRA_OPT_HYBRID_MIN_DOWN, int(down)), "mira_set_option")

    def down_slices(self, n: int = 0) -> None:
        """Reduction slices of the tcgen05 down kernel (0: chosen per step; 1..4 forced, at most ceil(ffn / 4096)).
        Set before the first wave of a step."""
        _check(mira_set_option(self._ctx, MIRA_OPT_DOWN_SLICES, int(n)), "mira_set_option")

    def test_wait_timeout(self) -> None:
        """Test hook: the next tcgen05 up/gate launch takes its time-out path in one CTA (see MIRA_OPT_TEST_WAIT_TIMEOUT)."""
        _check(mira_set_option(self._ctx, MIRA_OPT_TEST_WAIT_TIMEOUT, 1), "mira_set_option")

    def profile(self, enable: bool) -> None:
        _check(mira_profile(self._ctx, int(enable)), "mira_profile")

    def profile_read(self) -> dict:
        """{kernel class: (total ms, launches)} of the launches recorded since the last read."""
        n = len(KERNEL_CLASSES)
        ms, cnt = (C.c_float * n)(), (C.c_int64 * n)()
        _check(mira_profile_read(self._ctx, ms, cnt), "mira_profile_read")
        return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(KERNEL_CLASSES) if cnt[i]}

    @property
    def kernel_launches(self) -> int:
        return int(mira_kernel_launches(self._ctx))


def predict_noalloc(hidden, pred_w, pred_b=None, k_pred=2, pooled=None, ids=None, stream=None):
    """mira_predict_noalloc on caller-provided tensors. No context and no workspace are involved; if
    `pooled` / `ids` are given they are used as the outputs, so the call itself allocates nothing."""
    T, Cc = hidden.shape
    E = pred_w.shape[0]
    if pooled is None:
        pooled = torch.empty(E, dtype=torch.float32, device=hidden.device)
    if ids is None and k_pred > 0:
        ids = torch.empty(k_pred, dtype=torch.int32, device=hidden.device)
    _check(mira_predict_noalloc(_ptr(hidden), T, Cc, _ptr(pred_w), _ptr(pred_b), E, _ptr(pooled),
                                _ptr(ids) if k_pred > 0 else None, k_pred, _stream(stream)), "mira_predict_noalloc")
    return pooled, ids


def residual_rmsnorm(x: torch.Tensor, moe_out: torch.Tensor, eps: float = 1e-6, out=None, stream=None) -> torch.Tensor:
    """Harness glue: rmsnorm(x + moe_out) without learned scale, fp32 inside, bf16 out."""
    assert x.dtype == moe_out.dtype == torch.bfloat16 and x.shape == moe_out.shape and x.is_contiguous() and moe_out.is_contiguous()
    if out is None:
        out = torch.empty_like(x)
    _check(mira_residual_rmsnorm(_ptr(x), _ptr(moe_out), x.shape[0], x.shape[1], eps, _ptr(out), _stream(stream)),
           "mira_residual_rmsnorm")
    return out


def slot_table(blobs: torch.Tensor) -> torch.Tensor:
    """Device array of slot base pointers for a [n_slots, expert_bytes] uint8 tensor."""
    base, stride = blobs.data_ptr(), blobs.stride(0)
    return torch.tensor([base + i * stride for i in range(blobs.shape[0])], dtype=torch.int64, device=blobs.device)


class NativeLayerCache:
    """The library's cache bookkeeping object (mira_cache_*) behind the interface of cache.LayerCache, so either
    can drive the stack harness. Marshalling only: every decision is taken inside the library."""

    def __init__(self, n_routed: int, n_shared: int, hot, n_stage: int):
        from .cache import CacheStats, Wave
        self._Stats, self._Wave = CacheStats, Wave
        self.n_routed, self.n_shared, self.n_stage, self.n_hot = n_routed, n_shared, n_stage, len(hot)
        self.n = n_routed + n_shared
        self.n_slots = n_shared + self.n_hot + n_stage
        self.stage_first = n_shared + self.n_hot
        self._h = C.c_void_p()
        arr = (C.c_int32 * max(len(hot), 1))(*hot)
        _check(mira_cache_create(n_routed, n_shared, arr, len(hot), n_stage, C.byref(self._h)), "mira_cache_create")
        self.swaps_done = 0
        self._bufs = None
        self.win_tokens = 0                 # mirrors the library's window length (reset by each rebalancing pass)

    def close(self) -> None:
        if getattr(self, "_h", None) and mira_cache_destroy is not None:
            mira_cache_destroy(self._h)
            self._h = None

    __del__ = close

    def slot_map(self) -> list[int]:
        m = (C.c_int32 * self.n)()
        _check(mira_cache_slot_map(self._h, m), "mira_cache_slot_map")
        return list(m)

    def resident(self, e: int) -> bool:
        return self.slot_map()[e] >= 0

    def prefetch(self, predicted) -> list[tuple[int, int]]:
        predicted = list(predicted)
        p = (C.c_int32 * max(len(predicted), 1))(*predicted)
        oe, os_ = (C.c_int32 * self.n_stage)(), (C.c_int32 * self.n_stage)()
        n = mira_cache_prefetch(self._h, p, len(predicted), oe, os_)
        if n < 0:
            raise MiraError(MIRA_ERR_INVALID_ARG, "mira_cache_prefetch")
        return [(oe[i], os_[i]) for i in range(n)]

    def plan(self, counts) -> list:
        n = self.n
        assert len(counts) == n
        if self._bufs is None:                                             # reused by every call
            max_waves = 1 + (n + self.n_stage - 1) // self.n_stage
            self._bufs = ((C.c_int32 * n)(), (C.c_int32 * n)(), (C.c_int32 * n)(), (C.c_int32 * (n * max_waves))(), max_waves)
        c, wave_of, copy_slot, maps, max_waves = self._bufs
        c[:] = counts
        nw = mira_cache_plan(self._h, c, wave_of, copy_slot, maps, max_waves)
        if nw < 0:
            raise MiraError(MIRA_ERR_INVALID_ARG, "mira_cache_plan")
        waves = [self._Wave([], [], maps[w * n:(w + 1) * n]) for w in range(nw)]
        for e, (w, s) in enumerate(zip(wave_of[:], copy_slot[:])):
            if w >= 0:
                waves[w].experts.append(e)
                if s >= 0:
                    waves[w].copies.append((e, s))
        return waves

    def layer_done(self, n_tokens: int = 0) -> None:
        mira_cache_layer_done(self._h, n_tokens)
        self.win_tokens += n_tokens

    def rebalance(self, max_swaps: int = 2, miss_weight: float = 2.0, margin: float = 1.25):
        ev, pr, sl = ((C.c_int32 * max(max_swaps, 1))() for _ in range(3))
        n = mira_cache_rebalance(self._h, max_swaps, miss_weight, margin, ev, pr, sl)
        if n < 0:
            raise MiraError(MIRA_ERR_INVALID_ARG, "mira_cache_rebalance")
        self.swaps_done += n
        self.win_tokens = 0
        return [(ev[i], pr[i], sl[i]) for i in range(n)]

    @property
    def stats(self):
        out = (C.c_int64 * 11)()
        mira_cache_stats(self._h, out)
        return self._Stats(*list(out))

    def reset_stats(self) -> None:
        mira_cache_stats_reset(self._h)


class NativeStack:
    """mira_stack_* behind a small class: the library's layer-step runtime (predictor call, routing, prefetch and
    on-demand staging, waves, rebalancing) over caller-owned pinned host blobs and device slot memory."""

    def __init__(self, m: Mira, host_blobs: torch.Tensor, slot_mem: torch.Tensor, hot, n_hot: int, n_stage: int,
                 k_pred: int, side_stream, rebalance_every: int = 0, max_swaps: int = 2, miss_weight: float = 2.0,
                 margin: float = 1.25, stream=None):
        """host_blobs [L, E + n_shared, expert_bytes] pinned uint8; slot_mem [L, n_shared + n_hot + n_stage,
        expert_bytes] CUDA uint8; hot: L lists of n_hot expert ids."""
        from .cache import CacheStats
        self._Stats = CacheStats
        L = host_blobs.shape[0]
        assert host_blobs.is_pinned() and slot_mem.is_cuda and slot_mem.shape[0] == L
        assert host_blobs.shape[2] == m.expert_bytes == slot_mem.shape[2]
        assert slot_mem.shape[1] == m.ns + n_hot + n_stage and len(hot) == L and all(len(h) == n_hot for h in hot)
        self.m, self.L, self.k_pred = m, L, k_pred
        self.cfg = mira_stack_config(L, n_hot, n_stage, k_pred, rebalance_every, max_swaps, miss_weight, margin)
        nbytes = mira_stack_scratch_bytes(m._ctx, C.byref(self.cfg))
        if nbytes == 0:
            raise MiraError(MIRA_ERR_INVALID_ARG, "mira_stack_scratch_bytes")
        self.scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=m.device)
        base = (self.scratch.data_ptr() + 255) // 256 * 256
        self._keep = (host_blobs, slot_mem, side_stream)
        hp = (C.c_void_p * L)(*[host_blobs[l].data_ptr() for l in range(L)])
        sp = (C.c_void_p * L)(*[slot_mem[l].data_ptr() for l in range(L)])
        flat = [e for h in hot for e in h]
        ha = (C.c_int32 * max(len(flat), 1))(*flat)
        self._h = C.c_void_p()
        _check(mira_stack_create(m._ctx, C.byref(self.cfg), hp, sp, ha, C.c_void_p(base), nbytes,
                                 C.c_void_p(side_stream.cuda_stream), _stream(stream), C.byref(self._h)), "mira_stack_create")

    def close(self) -> None:
        if getattr(self, "_h", None) and mira_stack_destroy is not None:
            mira_stack_destroy(self._h)
            self._h = None

    __del__ = close

    def layer_step(self, layer: int, x, router_w, router_b, k: int, pred_w=None, pred_b=None, out=None, stream=None):
        T = x.shape[0]
        if out is None:
            out = torch.empty((T, self.m.C), dtype=self.m.out_dtype, device=self.m.device)
        _check(mira_stack_layer_step(self._h, layer, _ptr(x), T, _ptr(router_w), _ptr(router_b), k, _ptr(pred_w),
                                     _ptr(pred_b), _ptr(out), _stream(stream)), "mira_stack_layer_step")
        return out

    def stats(self):
        """(CacheStats summed over the layers, bytes staged, HOT swaps)."""
        v, b, sw = (C.c_int64 * 11)(), C.c_int64(), C.c_int64()
        _check(mira_stack_stats(self._h, v, C.byref(b), C.byref(sw)), "mira_stack_stats")
        return self._Stats(*list(v)), b.value, sw.value

    def reset_stats(self) -> None:
        mira_stack_stats_reset(self._h)

    def coverage(self):
        """(sums [L][k_pred], counts [L]) of Coverage@k per source layer."""
        kp = max(self.k_pred, 1)
        sums, n = (C.c_double * (self.L * kp))(), (C.c_int32 * self.L)()
        _check(mira_stack_coverage(self._h, sums, n), "mira_stack_coverage")
        return [[sums[l * kp + j] for j in range(self.k_pred)] for l in range(self.L)], list(n)

    def slot_map(self, layer: int):
        m = (C.c_int32 * (self.m.E + self.m.ns))()
        _check(mira_cache_slot_map(mira_stack_cache(self._h, layer), m), "mira_cache_slot_map")
        return list(m)
