"""ctypes binding of libl2pd.so: argument marshalling only.

PyTorch supplies device memory (tensors' data_ptr) and the current CUDA stream; every
arithmetic step runs inside the library's kernels.  The library must exist: importing this
module without it raises, there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libl2pd.so")

L2PD_F32, L2PD_BF16 = 0, 1
STATUS = {0: "L2PD_OK", -1: "L2PD_ERR_ARG", -2: "L2PD_ERR_SHAPE", -3: "L2PD_ERR_OOM", -4: "L2PD_ERR_CUDA",
          -5: "L2PD_ERR_TIMEOUT", -6: "L2PD_ERR_TOKEN_RANGE", -7: "L2PD_ERR_STATE"}


class L2pdError(RuntimeError):
    def __init__(self, status: int, msg: str = ""):
        self.status = status
        super().__init__("%s%s" % (STATUS.get(status, str(status)), (": " + msg) if msg else ""))


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("mask_id", C.c_int32), ("eot_id", C.c_int32), ("dtype", C.c_int32),
                ("block_len", C.c_int32), ("tau", C.c_float),
                ("use_filter", C.c_int32), ("use_eotp", C.c_int32), ("kv_cache_mode", C.c_int32),
                ("committed_conf_mode", C.c_int32), ("max_batch", C.c_int32), ("max_seq", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p),
                ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("w_gate", C.POINTER(C.c_void_p)), ("w_up", C.POINTER(C.c_void_p)),
                ("w_down", C.POINTER(C.c_void_p)),
                ("norm1", C.POINTER(C.c_void_p)), ("norm2", C.POINTER(C.c_void_p)),
                ("final_norm", C.c_void_p), ("lm_head", C.c_void_p), ("lm_head_bias", C.c_void_p),
                ("filt_w1", C.c_void_p), ("filt_b1", C.c_void_p), ("filt_w2", C.c_void_p), ("filt_b2", C.c_void_p)]


class TrainConfig(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("epochs", C.c_int32), ("batch_size", C.c_int32)]


class StepOut(C.Structure):
    _fields_ = [("d_conf", C.c_void_p), ("d_pred", C.c_void_p), ("d_p", C.c_void_p),
                ("d_unmask", C.c_void_p), ("d_logits", C.c_void_p),
                ("h_block", C.c_void_p), ("h_masks_left", C.c_void_p), ("h_l_eff", C.c_void_p),
                ("h_done", C.c_void_p), ("h_forced", C.c_void_p)]


EXPORTS = ["l2pd_init", "l2pd_state_reset", "l2pd_denoise_step", "l2pd_decode", "l2pd_num_active",
           "l2pd_state_tokens", "l2pd_state_masked", "l2pd_set_unmask_rule", "l2pd_set_filter", "l2pd_set_collect", "l2pd_collect_count", "l2pd_filter_train", "l2pd_filter_train_layers", "l2pd_set_capture", "l2pd_last_step_rows",
           "l2pd_launch_count", "l2pd_last_step_ms", "l2pd_profile_enable", "l2pd_profile_read", "l2pd_last_error", "l2pd_destroy",
           "l2pd_gemm_bf16", "l2pd_gemm_bf16_residual", "l2pd_gemm_bf16_swiglu", "l2pd_lm_head_bf16",
           "l2pd_lm_head_scratch_elems", "l2pd_attention_bf16", "l2pd_lm_head_bf16_static",
           "l2pd_set_chain", "l2pd_chain_trace_enable", "l2pd_chain_trace_read", "l2pd_debug_set_device_status"]


KINDS = ["embed", "gemm_qkv", "rope", "attention", "gemm_o", "rmsnorm", "gemm_gate_up", "gemm_down",
         "final_norm", "lm_head", "decide", "other", "gemm_chain"]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("libl2pd.so is missing at %s: build it with "
                          "`python -m paper_2509_25188_b200.build` (there is no fallback path)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.l2pd_init.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.c_int, C.POINTER(vp)]
    lib.l2pd_state_reset.argtypes = [vp, vp, vp, i32, i32, i32]
    lib.l2pd_denoise_step.argtypes = [vp, vp, C.POINTER(StepOut)]
    lib.l2pd_decode.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.l2pd_num_active.argtypes = [vp]
    lib.l2pd_state_tokens.argtypes = [vp]
    lib.l2pd_state_tokens.restype = vp
    lib.l2pd_state_masked.argtypes = [vp]
    lib.l2pd_state_masked.restype = vp
    lib.l2pd_set_capture.argtypes = [vp, vp, i64]
    lib.l2pd_set_unmask_rule.argtypes = [vp, vp, i32, f32, vp, i32, i32]
    lib.l2pd_set_filter.argtypes = [vp, i32, vp, vp]
    lib.l2pd_set_collect.argtypes = [vp, vp, vp, i64]
    lib.l2pd_collect_count.argtypes = [vp]
    lib.l2pd_collect_count.restype = i64
    lib.l2pd_filter_train.argtypes = [vp, i32, i64, vp, vp, vp, vp, vp, vp, C.POINTER(TrainConfig), vp]
    lib.l2pd_filter_train_layers.argtypes = [vp, i32, i32, i64, vp, vp, vp, vp, C.POINTER(TrainConfig), vp]
    lib.l2pd_last_step_rows.argtypes = [vp]
    lib.l2pd_launch_count.argtypes = [vp]
    lib.l2pd_launch_count.restype = i64
    lib.l2pd_last_step_ms.argtypes = [vp]
    lib.l2pd_last_step_ms.restype = f32
    lib.l2pd_profile_enable.argtypes = [vp, C.c_uint32]
    lib.l2pd_profile_read.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.l2pd_last_error.argtypes = [vp]
    lib.l2pd_last_error.restype = C.c_char_p
    lib.l2pd_destroy.argtypes = [vp]
    lib.l2pd_destroy.restype = None
    lib.l2pd_gemm_bf16.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32]
    lib.l2pd_gemm_bf16_residual.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32]
    lib.l2pd_gemm_bf16_swiglu.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32]
    lib.l2pd_lm_head_bf16.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, i32]
    lib.l2pd_lm_head_scratch_elems.argtypes = [i32, i32]
    lib.l2pd_lm_head_scratch_elems.restype = i64
    lib.l2pd_lm_head_bf16_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, i32]
    lib.l2pd_attention_bf16.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i64, i64, i64, i32, i32]
    lib.l2pd_debug_set_device_status.argtypes = [vp, vp, i32]
    lib.l2pd_set_chain.argtypes = [vp, i32]
    lib.l2pd_chain_trace_enable.argtypes = [vp, i32]
    lib.l2pd_chain_trace_read.argtypes = [vp, vp, i64, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.l2pd_chain_trace_read.restype = i64
    return lib


lib = _load()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, ctx=None):
    if status != 0:
        msg = lib.l2pd_last_error(ctx).decode()
        raise L2pdError(status, msg)


def to_device(arr: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy -> device tensor; uint16 arrays are bf16 bit patterns."""
    if arr.dtype == np.uint16:
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).to(device)


def _ptr_array(tensors):
    arr = (C.c_void_p * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        arr[i] = t.data_ptr()
    return arr


class Decoder:
    """Owns an l2pd context and the device copies of the weights it borrows."""

    def __init__(self, shape, weights: Dict[str, object], filt: Optional[Dict[str, np.ndarray]], *,
                 block_len: int, tau: float = 0.96, use_filter: bool = True, use_eotp: bool = True,
                 kv_cache: bool = False, committed_conf_mode: int = 0, max_batch: int = 1,
                 max_seq: int = 512, lm_head_bias: Optional[np.ndarray] = None, device: int = 0):
        torch.cuda.set_device(device)
        dev = "cuda:%d" % device
        self.shape = shape
        self.block_len = block_len
        self.device = device
        self._keep = []
        up = lambda a: self._hold(a if isinstance(a, torch.Tensor) else to_device(a, dev))
        layers = weights["layers"]
        names = ["wqkv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2"]
        per = {n: [up(l[n]) for l in layers] for n in names}
        self._arrays = {n: _ptr_array(per[n]) for n in names}
        w = Weights()
        w.tok_emb = up(weights["tok_emb"]).data_ptr()
        w.lm_head = up(weights["lm_head"]).data_ptr()
        w.final_norm = up(weights["final_norm"]).data_ptr()
        w.lm_head_bias = up(lm_head_bias).data_ptr() if lm_head_bias is not None else None
        for n in names:
            setattr(w, n, C.cast(self._arrays[n], C.POINTER(C.c_void_p)))
        if filt is not None:
            w.filt_w1, w.filt_b1 = up(filt["w1"]).data_ptr(), up(filt["b1"]).data_ptr()
            w.filt_w2, w.filt_b2 = up(filt["w2"]).data_ptr(), up(filt["b2"]).data_ptr()
        cfg = Config(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads,
                     head_dim=shape.head_dim, d_ff=shape.d_ff, vocab=shape.vocab, rms_eps=shape.rms_eps,
                     rope_theta=shape.rope_theta, mask_id=shape.mask_id, eot_id=shape.eot_id,
                     dtype=L2PD_BF16 if shape.dtype == "bf16" else L2PD_F32, block_len=block_len, tau=tau,
                     use_filter=int(use_filter and filt is not None), use_eotp=int(use_eotp),
                     kv_cache_mode=int(kv_cache), committed_conf_mode=committed_conf_mode,
                     max_batch=max_batch, max_seq=max_seq)
        self.cfg = cfg
        ctx = C.c_void_p()
        _check(lib.l2pd_init(C.byref(cfg), C.byref(w), device, C.byref(ctx)))
        self.ctx = ctx
        self.B = self.P = self.G = 0
        self._prompts = None

    def _hold(self, t: torch.Tensor) -> torch.Tensor:
        self._keep.append(t)
        return t

    def close(self):
        if getattr(self, "ctx", None):
            lib.l2pd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the three calls of the boundary -------------------------------------------------------
    def state_reset(self, prompts, G: int):
        p = prompts if isinstance(prompts, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(prompts))
        p = p.to("cuda:%d" % self.device, torch.int32).contiguous()
        self._prompts = p
        self.B, self.P, self.G = int(p.shape[0]), int(p.shape[1]), int(G)
        _check(lib.l2pd_state_reset(self.ctx, _stream(), p.data_ptr(), self.B, self.P, self.G), self.ctx)

    def denoise_step(self, want_logits: bool = False, outputs: bool = True) -> Optional[dict]:
        if not outputs:
            _check(lib.l2pd_denoise_step(self.ctx, _stream(), None), self.ctx)
            return None
        B, s, V = self.B, self.block_len, self.shape.vocab
        dev = "cuda:%d" % self.device
        t = {"conf": torch.zeros(B, s, device=dev), "pred": torch.full((B, s), -1, dtype=torch.int32, device=dev),
             "p": torch.zeros(B, s, device=dev), "unmask": torch.zeros(B, s, dtype=torch.uint8, device=dev)}
        if want_logits:
            t["logits"] = torch.zeros(B, s, V, device=dev)
        h = {k: np.full(B, -1, np.int32) for k in ("block", "masks_left", "l_eff", "done", "forced")}
        o = StepOut(d_conf=t["conf"].data_ptr(), d_pred=t["pred"].data_ptr(), d_p=t["p"].data_ptr(),
                    d_unmask=t["unmask"].data_ptr(), d_logits=t["logits"].data_ptr() if want_logits else None,
                    h_block=h["block"].ctypes.data, h_masks_left=h["masks_left"].ctypes.data,
                    h_l_eff=h["l_eff"].ctypes.data, h_done=h["done"].ctypes.data, h_forced=h["forced"].ctypes.data)
        _check(lib.l2pd_denoise_step(self.ctx, _stream(), C.byref(o)), self.ctx)
        out = {k: v.cpu().numpy() for k, v in t.items()}
        out.update(h)
        return out

    def state_reset_device(self, d_prompts: torch.Tensor, G: int):
        """state_reset on a caller-owned device tensor int32 [B, P] (no copy, no allocation)."""
        self.B, self.P, self.G = int(d_prompts.shape[0]), int(d_prompts.shape[1]), int(G)
        _check(lib.l2pd_state_reset(self.ctx, _stream(), d_prompts.data_ptr(), self.B, self.P, self.G), self.ctx)

    def denoise_step_host(self) -> dict:
        """One step; returns only the per-sequence host record (no device outputs)."""
        if getattr(self, "_hrec", None) is None or len(self._hrec["done"]) != self.B:
            self._hrec = {k: np.full(self.B, -1, np.int32) for k in ("block", "masks_left", "l_eff", "done", "forced")}
        h = self._hrec
        o = StepOut(h_block=h["block"].ctypes.data, h_masks_left=h["masks_left"].ctypes.data,
                    h_l_eff=h["l_eff"].ctypes.data, h_done=h["done"].ctypes.data, h_forced=h["forced"].ctypes.data)
        _check(lib.l2pd_denoise_step(self.ctx, _stream(), C.byref(o)), self.ctx)
        return h

    def denoise_step_into(self, d_conf: torch.Tensor, d_pred: torch.Tensor, d_unmask: torch.Tensor):
        """One step writing conf / pred / unmask [B, s] into caller-owned device tensors."""
        o = StepOut(d_conf=d_conf.data_ptr(), d_pred=d_pred.data_ptr(), d_unmask=d_unmask.data_ptr())
        _check(lib.l2pd_denoise_step(self.ctx, _stream(), C.byref(o)), self.ctx)

    def decode(self, prompts, G: int):
        """Returns (tokens [B,G] int32 numpy, out_len [B], steps [B], total_steps)."""
        p = prompts if isinstance(prompts, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(prompts))
        p = p.to("cuda:%d" % self.device, torch.int32).contiguous()
        B, P = int(p.shape[0]), int(p.shape[1])
        self.B, self.P, self.G = B, P, int(G)
        out = torch.empty(B, G, dtype=torch.int32, device=p.device)
        out_len = np.zeros(B, np.int32)
        steps = np.zeros(B, np.int32)
        total = C.c_int32(0)
        _check(lib.l2pd_decode(self.ctx, _stream(), p.data_ptr(), B, P, int(G), out.data_ptr(),
                               out_len.ctypes.data, steps.ctypes.data, C.addressof(total)), self.ctx)
        return out.cpu().numpy(), out_len, steps, int(total.value)

    def decode_device(self, d_prompts: torch.Tensor, G: int, d_out: torch.Tensor):
        """As decode, with caller-provided device tensors (nothing allocated, no copies)."""
        B, P = int(d_prompts.shape[0]), int(d_prompts.shape[1])
        self.B, self.P, self.G = B, P, int(G)
        out_len = np.zeros(B, np.int32)
        steps = np.zeros(B, np.int32)
        total = C.c_int32(0)
        _check(lib.l2pd_decode(self.ctx, _stream(), d_prompts.data_ptr(), B, P, int(G), d_out.data_ptr(),
                               out_len.ctypes.data, steps.ctypes.data, C.addressof(total)), self.ctx)
        return out_len, steps, int(total.value)

    RULES = {"filter": 0, "confidence": 1, "egp": 2}

    def set_unmask_rule(self, rule: str, conf_threshold: float = 0.9, reference=None):
        """rule: "filter" | "confidence" | "egp" (reference: int ids [rows, G], kept alive here)."""
        ref = None
        if rule == "egp":
            r = reference if isinstance(reference, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(reference))
            ref = r.to("cuda:%d" % self.device, torch.int32).contiguous()
            if ref.dim() != 2:
                raise ValueError("reference answers must be [rows, G]")
        _check(lib.l2pd_set_unmask_rule(self.ctx, _stream(), self.RULES[rule], float(conf_threshold),
                                        ref.data_ptr() if ref is not None else None,
                                        int(ref.shape[0]) if ref is not None else 0,
                                        int(ref.shape[1]) if ref is not None else 0), self.ctx)
        self._reference = ref

    def set_filter_layers(self, layers):
        """layers: list of (W [s, s], b [s]) numpy arrays, 1 to 4 of them; [] restores the init-time filter."""
        dev = "cuda:%d" % self.device
        ws = [torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).to(dev) for w, _ in layers]
        bs = [torch.from_numpy(np.ascontiguousarray(b, dtype=np.float32)).to(dev) for _, b in layers]
        n = len(layers)
        pw = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in ws])
        pb = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in bs])
        _check(lib.l2pd_set_filter(self.ctx, n, pw, pb), self.ctx)
        self._filter_layers = (ws, bs)

    def set_collect(self, capacity: int):
        """Starts (capacity > 0) or stops (0) collecting Algorithm 1's samples; returns the device sinks."""
        if capacity <= 0:
            _check(lib.l2pd_set_collect(self.ctx, None, None, 0), self.ctx)
            self._sink = None
            return None
        dev = "cuda:%d" % self.device
        c = torch.zeros(capacity, self.block_len, device=dev)
        y = torch.zeros(capacity, self.block_len, dtype=torch.uint8, device=dev)
        _check(lib.l2pd_set_collect(self.ctx, c.data_ptr(), y.data_ptr(), capacity), self.ctx)
        self._sink = (c, y)
        return c, y

    @property
    def collect_count(self) -> int:
        return int(lib.l2pd_collect_count(self.ctx))

    def debug_set_device_status(self, code: int):
        """Test hook: presets the device status word (what a kernel's exhausted bounded wait would leave)."""
        _check(lib.l2pd_debug_set_device_status(self.ctx, _stream(), int(code)), self.ctx)

    # ---- chained launches ------------------------------------------------------------------------
    def set_chain(self, mode):
        """0 / False: one launch per projection (the default); 1 / True: one persistent launch per layer where the step's
        shapes allow; 2: the chained form's tiling in single launches (bit-identical to 1, for comparisons)."""
        _check(lib.l2pd_set_chain(self.ctx, int(mode)), self.ctx)

    def chain_trace_enable(self, enable: bool = True):
        _check(lib.l2pd_chain_trace_enable(self.ctx, int(bool(enable))), self.ctx)

    def chain_trace(self) -> Optional[np.ndarray]:
        """Stamps of the last step's chained launches, uint64 [launch, phase slot, 4 (opened, first / last accumulator ready, finished), CTA] in ns."""
        nl, nph, nc = C.c_int32(0), C.c_int32(0), C.c_int32(0)
        n = lib.l2pd_chain_trace_read(self.ctx, None, 0, C.byref(nl), C.byref(nph), C.byref(nc))
        if n <= 0:
            return None
        out = np.zeros(n, np.uint64)
        got = lib.l2pd_chain_trace_read(self.ctx, out.ctypes.data, n, C.byref(nl), C.byref(nph), C.byref(nc))
        if got != n:
            raise L2pdError(-4, "chain trace read failed")
        return out.reshape(nl.value, nph.value, 4, nc.value)

    # ---- state and instrumentation -------------------------------------------------------------
    @property
    def num_active(self) -> int:
        return lib.l2pd_num_active(self.ctx)

    def tokens(self) -> np.ndarray:
        L = self.P + self.G
        v = _DeviceView(lib.l2pd_state_tokens(self.ctx), (self.B, L), "<i4")
        return torch.as_tensor(v, device="cuda:%d" % self.device).cpu().numpy()

    def masked(self) -> np.ndarray:
        v = _DeviceView(lib.l2pd_state_masked(self.ctx), (self.B, self.G), "|u1")
        return torch.as_tensor(v, device="cuda:%d" % self.device).cpu().numpy().astype(bool)

    def set_capture(self, tensor: Optional[torch.Tensor]):
        if tensor is None:
            _check(lib.l2pd_set_capture(self.ctx, None, 0), self.ctx)
        else:
            _check(lib.l2pd_set_capture(self.ctx, tensor.data_ptr(), tensor.stride(0)), self.ctx)

    def profile_enable(self, kinds):
        mask = 0
        for k in kinds:
            mask |= 1 << KINDS.index(k)
        _check(lib.l2pd_profile_enable(self.ctx, mask), self.ctx)

    def profile_read(self) -> dict:
        out = {}
        for i, k in enumerate(KINDS):
            ms, n = C.c_double(0), C.c_int64(0)
            _check(lib.l2pd_profile_read(self.ctx, i, C.byref(ms), C.byref(n)), self.ctx)
            if n.value:
                out[k] = (ms.value, n.value)
        return out

    @property
    def last_step_rows(self) -> int:
        return lib.l2pd_last_step_rows(self.ctx)

    @property
    def launch_count(self) -> int:
        return lib.l2pd_launch_count(self.ctx)

    @property
    def last_step_ms(self) -> float:
        return lib.l2pd_last_step_ms(self.ctx)


class _DeviceView:
    """View of library-owned device memory (CUDA array interface); callers only read it."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr,
                                         "data": (int(ptr), False), "version": 2}


# ---- stand-alone kernels -------------------------------------------------------------------------

def gemm_bf16(A: torch.Tensor, W: torch.Tensor, tile_n: int = 0) -> torch.Tensor:
    M, K = A.shape
    N = W.shape[0]
    Cc = torch.empty(M, N, dtype=torch.bfloat16, device=A.device)
    _check(lib.l2pd_gemm_bf16(_stream(), A.data_ptr(), W.data_ptr(), Cc.data_ptr(), M, N, K, tile_n, 1))
    return Cc


def gemm_bf16_residual(A: torch.Tensor, W: torch.Tensor, X: torch.Tensor, tile_n: int = 0) -> torch.Tensor:
    M, K = A.shape
    N = W.shape[0]
    _check(lib.l2pd_gemm_bf16_residual(_stream(), A.data_ptr(), W.data_ptr(), X.data_ptr(), M, N, K, tile_n, 1))
    return X


def gemm_bf16_swiglu(A: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor, tile_n: int = 0) -> torch.Tensor:
    M, K = A.shape
    F = Wg.shape[0]
    H = torch.empty(M, F, dtype=torch.bfloat16, device=A.device)
    _check(lib.l2pd_gemm_bf16_swiglu(_stream(), A.data_ptr(), Wg.data_ptr(), Wu.data_ptr(), H.data_ptr(),
                                     M, F, K, tile_n, 1))
    return H


def lm_head_bf16(A: torch.Tensor, W: torch.Tensor, bias: Optional[torch.Tensor] = None, want_logits=False):
    R, K = A.shape
    V = W.shape[0]
    scratch = torch.empty(lib.l2pd_lm_head_scratch_elems(R, V), dtype=torch.float32, device=A.device)
    pred = torch.empty(R, dtype=torch.int32, device=A.device)
    conf = torch.empty(R, dtype=torch.float32, device=A.device)
    logits = torch.empty(R, V, dtype=torch.float32, device=A.device) if want_logits else None
    _check(lib.l2pd_lm_head_bf16(_stream(), A.data_ptr(), W.data_ptr(), bias.data_ptr() if bias is not None else None,
                                 R, V, K, scratch.data_ptr(), pred.data_ptr(), conf.data_ptr(),
                                 logits.data_ptr() if want_logits else None, 1))
    return pred, conf, logits


def lm_head_bf16_static(A: torch.Tensor, W: torch.Tensor, bias: Optional[torch.Tensor], pred: torch.Tensor,
                        conf: torch.Tensor):
    """LM head + confidence head through the entry point that allocates nothing: for callers whose
    device memory is handed out by their own arena (or is fully committed) and who therefore pass
    only inputs and outputs; the scratch is a fixed array inside the library (R <= 128, V <= 131072).
    `pred` (int32 [R]) and `conf` (float32 [R]) are caller-owned device tensors."""
    R, K = A.shape
    V = W.shape[0]
    _check(lib.l2pd_lm_head_bf16_static(_stream(), A.data_ptr(), W.data_ptr(),
                                        bias.data_ptr() if bias is not None else None, R, V, K,
                                        pred.data_ptr(), conf.data_ptr(), 1))
    return pred, conf


def attention_bf16(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, H: int, dh: int, impl: int = 0) -> torch.Tensor:
    """impl 0: tensor-memory kernel where it applies (dh 128), 1: the warp-level kernel."""
    Tq, Tk = q.shape[0], k.shape[0]
    out = torch.empty(Tq, H * dh, dtype=torch.bfloat16, device=q.device)
    _check(lib.l2pd_attention_bf16(_stream(), q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                   Tq, Tk, H, dh, q.stride(0), k.stride(0), out.stride(0), impl, 1))
    return out


def filter_train(filt: Dict[str, np.ndarray], C_in, Y_in, epochs: int, lr: float = 1e-3, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.01, batch_size: int = 0,
                 device: int = 0):
    """Algorithm 1, stage 2 on the GPU.  C_in [N, s] float, Y_in [N, s] 0/1 (numpy or device tensors).
    Returns (trained filter as numpy fp32 arrays, losses [updates])."""
    dev = "cuda:%d" % device
    torch.cuda.set_device(device)
    tc = (C_in if isinstance(C_in, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(C_in))).to(dev, torch.float32).contiguous()
    ty = (Y_in if isinstance(Y_in, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(Y_in))).to(dev, torch.uint8).contiguous()
    N, s = int(tc.shape[0]), int(tc.shape[1])
    p = {k: torch.from_numpy(np.ascontiguousarray(filt[k], dtype=np.float32)).to(dev) for k in ("w1", "b1", "w2", "b2")}
    bs = N if batch_size <= 0 else batch_size
    losses = np.zeros(max(epochs * (-(-N // bs)), 1), np.float32)
    cfg = TrainConfig(lr, beta1, beta2, eps, weight_decay, epochs, batch_size)
    _check(lib.l2pd_filter_train(_stream(), s, N, tc.data_ptr(), ty.data_ptr(), p["w1"].data_ptr(), p["b1"].data_ptr(),
                                 p["w2"].data_ptr(), p["b2"].data_ptr(), C.byref(cfg), losses.ctypes.data), None)
    return {k: v.cpu().numpy() for k, v in p.items()}, losses[: epochs * (-(-N // bs))]


def filter_train_layers(layers, C_in, Y_in, epochs: int, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999,
                        eps: float = 1e-8, weight_decay: float = 0.01, batch_size: int = 0, device: int = 0):
    """filter_train for a filter given as a list of 1 to 4 (W [s, s], b [s]) layers; returns (layers, losses)."""
    dev = "cuda:%d" % device
    torch.cuda.set_device(device)
    tc = (C_in if isinstance(C_in, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(C_in))).to(dev, torch.float32).contiguous()
    ty = (Y_in if isinstance(Y_in, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(Y_in))).to(dev, torch.uint8).contiguous()
    N, s = int(tc.shape[0]), int(tc.shape[1])
    ws = [torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).to(dev) for w, _ in layers]
    bs_ = [torch.from_numpy(np.ascontiguousarray(b_, dtype=np.float32)).to(dev) for _, b_ in layers]
    n = len(layers)
    pw = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in ws])
    pb = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in bs_])
    bsz = N if batch_size <= 0 else batch_size
    updates = epochs * (-(-N // bsz))
    losses = np.zeros(max(updates, 1), np.float32)
    cfg = TrainConfig(lr, beta1, beta2, eps, weight_decay, epochs, batch_size)
    _check(lib.l2pd_filter_train_layers(_stream(), s, n, N, tc.data_ptr(), ty.data_ptr(), pw, pb, C.byref(cfg),
                                        losses.ctypes.data), None)
    return [(w.cpu().numpy(), b_.cpu().numpy()) for w, b_ in zip(ws, bs_)], losses[:updates]
