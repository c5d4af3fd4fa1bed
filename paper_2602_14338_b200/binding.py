"""ctypes binding of libaero_b200.so: argument marshalling only.

Every function here has the name and argument order of its C counterpart in
include/aero.h.  Tensors are torch CUDA tensors used purely as device buffers;
the binding passes their data pointers and checks dtype/shape/contiguity.  There
is no fallback: if the library is missing or has no CUDA device, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AERO_B200_LIB") or os.path.join(_HERE, "libaero_b200.so")

AERO_UNIFORM_MASK, AERO_UNIFORM_BAYES = 0, 1
AERO_STATS_KEPT, AERO_STATS_ALL = 0, 1
AERO_TOKEN_MEAN, AERO_SEQ_MEAN = 0, 1
AERO_DENOM_SURVIVING, AERO_DENOM_ALL = 0, 1
AERO_BF16, AERO_FP32 = 0, 1
AERO_ST_BAD_TARGET, AERO_ST_BAD_OFFSETS, AERO_ST_BAD_REWARD, AERO_ST_EMPTY_ROLLOUT, AERO_ST_TIMEOUT = 1, 2, 4, 8, 16
AERO_ST_RANGE = 32

EXPORTS = [
    "aero_version", "aero_error_string", "aero_cfg_default", "aero_create", "aero_destroy",
    "aero_set_stream", "aero_last_status", "aero_group_workspace_bytes", "aero_group_stats",
    "aero_fwd_workspace_bytes", "aero_grpo_loss_fwd", "aero_bwd_workspace_bytes", "aero_grpo_loss_bwd",
    "aero_step_workspace_bytes", "aero_grpo_step_host", "aero_launch_count", "aero_group_stats_static",
    "aero_grpo_loss_reg_fwd", "aero_grpo_loss_reg_bwd", "aero_logprob_fwd",
    "aero_alloc_cfg_default", "aero_allocate_workspace_bytes", "aero_allocate_sim",
    "aero_fwd_bwd_workspace_bytes", "aero_grpo_loss_fwd_bwd", "aero_grpo_loss_kl_fwd_bwd", "aero_grpo_loss_reg_fwd_bwd",
    "aero_enable_kernel_timing", "aero_kernel_timing_ms",
    "aero_set_tuning", "aero_finalize_weights", "aero_selftest_bounded_wait",
]


class AeroCfg(C.Structure):
    _fields_ = [
        ("uniform_policy", C.c_int32), ("rejection", C.c_int32), ("k_ratio", C.c_int32),
        ("rescue_S", C.c_int32), ("n_explore", C.c_int32), ("n_keep_uniform", C.c_int32),
        ("stats_over", C.c_int32), ("agg", C.c_int32), ("denom", C.c_int32),
        ("alpha0", C.c_float), ("beta0", C.c_float), ("eps_std", C.c_float),
        ("clip_lo", C.c_float), ("clip_hi", C.c_float),
        ("seed", C.c_uint64), ("dtype", C.c_int32), ("reject_high", C.c_int32),
        ("kl_beta", C.c_float), ("ent_coef", C.c_float),
    ]


class AeroAllocCfg(C.Structure):
    _fields_ = [("n_extra", C.c_int32), ("k_max", C.c_int32), ("n_max", C.c_int32), ("n_budget", C.c_int32)]


class AeroError(RuntimeError):
    pass


_lib = None


def load_library():
    """Load libaero_b200.so and declare the C signatures.  Raises if the file is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise AeroError(f"{LIB_PATH} not found: build it with `python -m paper_2602_14338_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    lib.aero_version.restype = C.c_int
    lib.aero_error_string.restype = C.c_char_p
    lib.aero_error_string.argtypes = [C.c_int]
    lib.aero_cfg_default.restype = None
    lib.aero_cfg_default.argtypes = [C.POINTER(AeroCfg)]
    lib.aero_create.argtypes = [C.POINTER(vp), C.c_int, vp]
    lib.aero_destroy.argtypes = [vp]
    lib.aero_set_stream.argtypes = [vp, vp]
    lib.aero_set_tuning.argtypes = [vp, C.c_char_p, C.c_int]
    lib.aero_selftest_bounded_wait.argtypes = [vp, C.c_uint32]
    lib.aero_last_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.aero_group_workspace_bytes.restype = sz
    lib.aero_group_workspace_bytes.argtypes = [i32, i32]
    lib.aero_group_stats.argtypes = [vp, C.POINTER(AeroCfg), i32, i32] + [vp] * 19 + [vp, sz]
    lib.aero_group_stats_static.argtypes = [vp, C.POINTER(AeroCfg), i32, i32] + [vp] * 19
    lib.aero_finalize_weights.argtypes = [vp, C.POINTER(AeroCfg), i32, i32, i64, vp, vp, vp]
    lib.aero_fwd_workspace_bytes.restype = sz
    lib.aero_fwd_workspace_bytes.argtypes = [i64, i32, i32, i32]
    lib.aero_grpo_loss_fwd.argtypes = [vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 13 + [C.c_int, vp, sz]
    lib.aero_bwd_workspace_bytes.restype = sz
    lib.aero_bwd_workspace_bytes.argtypes = [i64, i32, i32, i32, i64]
    lib.aero_grpo_loss_bwd.argtypes = ([vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 8 + [f32] +
                                       [vp, vp, C.c_int, vp, sz])
    lib.aero_grpo_loss_reg_fwd.argtypes = ([vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 15 +
                                           [C.c_int, vp, sz])
    lib.aero_grpo_loss_reg_bwd.argtypes = ([vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 10 + [f32] +
                                           [vp, vp, C.c_int, vp, sz])
    lib.aero_logprob_fwd.argtypes = [vp, C.POINTER(AeroCfg), i64, i32, i32] + [vp] * 6 + [vp, sz]
    lib.aero_alloc_cfg_default.restype = None
    lib.aero_alloc_cfg_default.argtypes = [C.POINTER(AeroAllocCfg)]
    lib.aero_allocate_workspace_bytes.restype = sz
    lib.aero_allocate_workspace_bytes.argtypes = [i32]
    lib.aero_allocate_sim.argtypes = [vp, C.POINTER(AeroCfg), C.POINTER(AeroAllocCfg), i32] + [vp] * 5 + [vp, sz]
    lib.aero_fwd_bwd_workspace_bytes.restype = sz
    lib.aero_fwd_bwd_workspace_bytes.argtypes = [i64, i32, i32, i32, i64]
    lib.aero_grpo_loss_fwd_bwd.argtypes = ([vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 13 + [f32] +
                                           [vp, vp, C.c_int, vp, sz])
    lib.aero_grpo_loss_kl_fwd_bwd.argtypes = ([vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 14 + [f32] +
                                              [vp, vp, C.c_int, vp, sz])
    lib.aero_grpo_loss_reg_fwd_bwd.argtypes = ([vp, C.POINTER(AeroCfg), i64, i32, i32, i32] + [vp] * 15 + [f32] +
                                               [vp, vp, C.c_int, vp, sz])
    lib.aero_enable_kernel_timing.argtypes = [vp, C.c_int]
    lib.aero_kernel_timing_ms.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int)]
    lib.aero_step_workspace_bytes.restype = sz
    lib.aero_step_workspace_bytes.argtypes = [i32, i32, i64, i32, i32, i64, i32]
    lib.aero_grpo_step_host.argtypes = ([vp, C.POINTER(AeroCfg), i32, i32, i64, i32, i32] + [vp] * 12 + [C.c_int] +
                                        [vp, vp, vp, vp, sz])
    lib.aero_launch_count.restype = C.c_int64
    lib.aero_launch_count.argtypes = [vp]
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != 0:
        msg = load_library().aero_error_string(rc).decode()
        raise AeroError(f"{what} failed: {msg} ({rc})")


def cfg_default(**over) -> AeroCfg:
    cfg = AeroCfg()
    load_library().aero_cfg_default(C.byref(cfg))
    for k, v in over.items():
        if not hasattr(cfg, k):
            raise AttributeError(k)
        setattr(cfg, k, v)
    return cfg


def alloc_cfg_default(**over) -> AeroAllocCfg:
    ac = AeroAllocCfg()
    load_library().aero_alloc_cfg_default(C.byref(ac))
    for k, v in over.items():
        if not hasattr(ac, k):
            raise AttributeError(k)
        setattr(ac, k, v)
    return ac


def _ptr(t, dtype=None, numel=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise AeroError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise AeroError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if numel is not None and t.numel() < numel:
        raise AeroError(f"{name} has {t.numel()} elements, needs {numel}")
    return t.data_ptr()


def _ptr_key(key, R):
    if key is None:
        return None
    if key.dtype not in (torch.int32, torch.uint32):
        raise AeroError("key must be a 32-bit integer tensor (its bits are read as unsigned)")
    return _ptr(key, None, R, "key")


class Context:
    """Owns an aero_ctx bound to a device and (borrowed) to the current torch stream."""

    def __init__(self, device=0, stream=None):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise AeroError("no CUDA device: this library has no CPU path")
        self.device = torch.device("cuda", device)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        self.stream = stream
        h = C.c_void_p()
        _check(self.lib.aero_create(C.byref(h), device, C.c_void_p(stream.cuda_stream)), "aero_create")
        self.h = h
        self._ws = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.aero_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream):
        self.stream = stream
        _check(self.lib.aero_set_stream(self.h, C.c_void_p(stream.cuda_stream)), "aero_set_stream")

    def set_tuning(self, vsplit=0, nsync=-1, rowscale=-1, gemm_sync=-1, gemm_pairs=-1, w_hint=-1, k_zigzag=-1):
        """aero_set_tuning for every setting: schedule choices of stage (b); the defaults let the library decide."""
        for name, value in (("vsplit", vsplit), ("nsync", nsync), ("rowscale", rowscale), ("gemm_sync", gemm_sync),
                            ("gemm_pairs", gemm_pairs), ("w_hint", w_hint), ("k_zigzag", k_zigzag)):
            _check(self.lib.aero_set_tuning(self.h, name.encode(), int(value)), f"aero_set_tuning({name})")

    def selftest_bounded_wait(self, limit_us=1000):
        """aero_selftest_bounded_wait: a wait that cannot complete must end with AERO_ST_TIMEOUT."""
        _check(self.lib.aero_selftest_bounded_wait(self.h, int(limit_us)), "aero_selftest_bounded_wait")

    def last_status(self) -> int:
        bits = C.c_uint32(0)
        _check(self.lib.aero_last_status(self.h, C.byref(bits)), "aero_last_status")
        return bits.value

    def workspace(self, nbytes: int):
        """A cached uint8 device buffer of at least nbytes (256-byte aligned by the torch allocator)."""
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.device)
        return self._ws

    # ---- stage (a) ------------------------------------------------------------------
    def group_workspace_bytes(self, P, R):
        return self.lib.aero_group_workspace_bytes(P, R)

    def group_stats(self, cfg, go, reward, cs, key=None, keep_in=None, alpha_in=None, beta_in=None, out=None):
        P, R = go.numel() - 1, reward.numel()
        dev = self.device
        o = out if out is not None else {}

        def buf(name, n, dt):
            if name not in o:
                o[name] = torch.empty(max(n, 1), dtype=dt, device=dev)
            return o[name]

        adv, w = buf("adv", R, torch.float32), buf("w", R, torch.float32)
        keep, gmask, cat = buf("keep", R, torch.uint8), buf("gmask", P, torch.uint8), buf("cat", P, torch.uint8)
        u, ao, bo = buf("u_tilde", P, torch.float32), buf("alpha_out", P, torch.float32), buf("beta_out", P, torch.float32)
        kid, kto = buf("kept_ids", R, torch.int32), buf("kept_tok_off", R + 1, torch.int64)
        cnt, met = buf("counters", 8, torch.int64), buf("metrics", 4, torch.float32)
        ws = self.workspace(self.group_workspace_bytes(P, R))
        rc = self.lib.aero_group_stats(
            self.h, C.byref(cfg), P, R, _ptr(go, torch.int32, P + 1, "go"), _ptr(reward, torch.float32, R, "reward"),
            _ptr(cs, torch.int64, R + 1, "cs"), _ptr_key(key, R),
            _ptr(keep_in, torch.uint8, R, "keep_in"), _ptr(alpha_in, torch.float32, P, "alpha_in"),
            _ptr(beta_in, torch.float32, P, "beta_in"), _ptr(adv), _ptr(w), _ptr(keep), _ptr(gmask), _ptr(cat),
            _ptr(u), _ptr(ao), _ptr(bo), _ptr(kid), _ptr(kto), _ptr(cnt), _ptr(met), ws.data_ptr(), ws.numel())
        _check(rc, "aero_group_stats")
        return o

    def finalize_weights(self, cfg, w, counters_local, counters_global, P_local, P_global):
        """aero_finalize_weights: rescale a shard's weights from its local to the batch-wide denominator."""
        R = w.numel()
        rc = self.lib.aero_finalize_weights(self.h, C.byref(cfg), R, P_local, P_global, _ptr(w, torch.float32, R, "w"),
                                            _ptr(counters_local, torch.int64, 8, "counters_local"),
                                            _ptr(counters_global, torch.int64, 8, "counters_global"))
        _check(rc, "aero_finalize_weights")
        return w

    GROUP_OUTPUTS = (("adv", "R", torch.float32), ("w", "R", torch.float32), ("keep", "R", torch.uint8),
                     ("gmask", "P", torch.uint8), ("cat", "P", torch.uint8), ("u_tilde", "P", torch.float32),
                     ("alpha_out", "P", torch.float32), ("beta_out", "P", torch.float32),
                     ("kept_ids", "R", torch.int32), ("kept_tok_off", "R1", torch.int64),
                     ("counters", "8", torch.int64), ("metrics", "4", torch.float32))

    def group_stats_static(self, cfg, go, reward, cs, out, key=None, keep_in=None, alpha_in=None, beta_in=None):
        """aero_group_stats_static: the results of group_stats with the scratch taken from the array
        that is part of the loaded library.  Nothing is allocated here either: `out` must already
        hold every output tensor (names and sizes as group_stats returns them), so a caller that
        cannot allocate at this point can still make the call."""
        P, R = go.numel() - 1, reward.numel()
        size = {"R": R, "P": P, "R1": R + 1, "8": 8, "4": 4}
        ptrs = []
        for name, n, dt in self.GROUP_OUTPUTS:
            if name not in out:
                raise AeroError(f"group_stats_static needs a preallocated '{name}' tensor")
            ptrs.append(_ptr(out[name], dt, size[n], name))
        rc = self.lib.aero_group_stats_static(
            self.h, C.byref(cfg), P, R, _ptr(go, torch.int32, P + 1, "go"), _ptr(reward, torch.float32, R, "reward"),
            _ptr(cs, torch.int64, R + 1, "cs"), _ptr_key(key, R),
            _ptr(keep_in, torch.uint8, R, "keep_in"), _ptr(alpha_in, torch.float32, P, "alpha_in"),
            _ptr(beta_in, torch.float32, P, "beta_in"), *ptrs)
        _check(rc, "aero_group_stats_static")
        return out

    # ---- stage (b) ------------------------------------------------------------------
    def fwd_workspace_bytes(self, T, d, V, R):
        return self.lib.aero_fwd_workspace_bytes(T, d, V, R)

    def bwd_workspace_bytes(self, T, d, V, R, chunk_tokens):
        return self.lib.aero_bwd_workspace_bytes(T, d, V, R, chunk_tokens)

    def grpo_loss_fwd(self, cfg, H, W, y, old_logp, cs, adv, w, keep, out=None, accumulate=False):
        T, d = H.shape
        V = W.shape[0]
        R = cs.numel() - 1
        dt = torch.bfloat16 if cfg.dtype == AERO_BF16 else torch.float32
        o = out if out is not None else {}
        for name in ("logp", "lse", "g"):
            if name not in o:
                o[name] = torch.empty(max(T, 1), dtype=torch.float32, device=self.device)
        if "loss" not in o:
            o["loss"] = torch.zeros(1, dtype=torch.float32, device=self.device)
        if "metrics" not in o:
            o["metrics"] = torch.zeros(4, dtype=torch.float32, device=self.device)
        ws = self.workspace(self.fwd_workspace_bytes(T, d, V, R))
        rc = self.lib.aero_grpo_loss_fwd(
            self.h, C.byref(cfg), T, d, V, R, _ptr(H, dt, T * d, "H"), _ptr(W, dt, V * d, "W"),
            _ptr(y, torch.int32, T, "y"), _ptr(old_logp, torch.float32, T, "old_logp"),
            _ptr(cs, torch.int64, R + 1, "cs"), _ptr(adv, torch.float32, R, "adv"), _ptr(w, torch.float32, R, "w"),
            _ptr(keep, torch.uint8, R, "keep"), _ptr(o["logp"]), _ptr(o["lse"]), _ptr(o["g"]), _ptr(o["loss"]),
            _ptr(o["metrics"]), 1 if accumulate else 0, ws.data_ptr(), ws.numel())
        _check(rc, "aero_grpo_loss_fwd")
        return o

    def grpo_loss_reg_fwd(self, cfg, H, W, y, old_logp, ref_logp, cs, adv, w, keep, out=None, accumulate=False,
                          entropy=True):
        """aero_grpo_loss_reg_fwd: the forward with Eq. 2's KL term (ref_logp not None) and the entropy
        bonus (entropy=True adds the per-row entropy output 'entropy')."""
        T, d = H.shape
        V = W.shape[0]
        R = cs.numel() - 1
        dt = torch.bfloat16 if cfg.dtype == AERO_BF16 else torch.float32
        o = out if out is not None else {}
        names = ("logp", "lse", "g", "entropy") if entropy else ("logp", "lse", "g")
        for name in names:
            if name not in o:
                o[name] = torch.empty(max(T, 1), dtype=torch.float32, device=self.device)
        if "loss" not in o:
            o["loss"] = torch.zeros(1, dtype=torch.float32, device=self.device)
        if "metrics" not in o:
            o["metrics"] = torch.zeros(4, dtype=torch.float32, device=self.device)
        ws = self.workspace(self.fwd_workspace_bytes(T, d, V, R))
        rc = self.lib.aero_grpo_loss_reg_fwd(
            self.h, C.byref(cfg), T, d, V, R, _ptr(H, dt, T * d, "H"), _ptr(W, dt, V * d, "W"),
            _ptr(y, torch.int32, T, "y"), _ptr(old_logp, torch.float32, T, "old_logp"),
            _ptr(ref_logp, torch.float32, T, "ref_logp"),
            _ptr(cs, torch.int64, R + 1, "cs"), _ptr(adv, torch.float32, R, "adv"), _ptr(w, torch.float32, R, "w"),
            _ptr(keep, torch.uint8, R, "keep"), _ptr(o["logp"]), _ptr(o["lse"]), _ptr(o["g"]),
            _ptr(o["entropy"]) if entropy else None, _ptr(o["loss"]),
            _ptr(o["metrics"]), 1 if accumulate else 0, ws.data_ptr(), ws.numel())
        _check(rc, "aero_grpo_loss_reg_fwd")
        return o

    def logprob_fwd(self, cfg, H, W, y, entropy=False, out=None):
        """aero_logprob_fwd: log-probs (and optionally entropies) of the target tokens of all T rows."""
        T, d = H.shape
        V = W.shape[0]
        dt = torch.bfloat16 if cfg.dtype == AERO_BF16 else torch.float32
        o = out if out is not None else {}
        names = ("logp", "lse", "entropy") if entropy else ("logp", "lse")
        for name in names:
            if name not in o:
                o[name] = torch.empty(max(T, 1), dtype=torch.float32, device=self.device)
        ws = self.workspace(self.fwd_workspace_bytes(T, d, V, 0))
        rc = self.lib.aero_logprob_fwd(
            self.h, C.byref(cfg), T, d, V, _ptr(H, dt, T * d, "H"), _ptr(W, dt, V * d, "W"),
            _ptr(y, torch.int32, T, "y"), _ptr(o["logp"]), _ptr(o["lse"]),
            _ptr(o["entropy"]) if entropy else None, ws.data_ptr(), ws.numel())
        _check(rc, "aero_logprob_fwd")
        return o

    def grpo_loss_reg_bwd(self, cfg, H, W, y, cs, keep, lse, g, entropy, w, grad_scale=1.0, dH=None, dW=None,
                          accumulate_dW=False, chunk_tokens=None, workspace=None, logp=None):
        """aero_grpo_loss_reg_bwd: the backward with the entropy term (entropy and w from the forward / group stage)."""
        T, d = H.shape
        V = W.shape[0]
        R = cs.numel() - 1
        dt = torch.bfloat16 if cfg.dtype == AERO_BF16 else torch.float32
        if dH is None:
            dH = torch.empty((max(T, 1), d), dtype=dt, device=self.device)[:T]
        if dW is None:
            dW = torch.empty((V, d), dtype=torch.float32, device=self.device)
        if workspace is None:
            if chunk_tokens is None:
                chunk_tokens = min(max(128, (T + 127) // 128 * 128), 2 * 148 * 128)
            workspace = self.workspace(self.bwd_workspace_bytes(T, d, V, R, chunk_tokens))
        rc = self.lib.aero_grpo_loss_reg_bwd(
            self.h, C.byref(cfg), T, d, V, R, _ptr(H, dt, T * d, "H"), _ptr(W, dt, V * d, "W"),
            _ptr(y, torch.int32, T, "y"), _ptr(cs, torch.int64, R + 1, "cs"), _ptr(keep, torch.uint8, R, "keep"),
            _ptr(lse, torch.float32, T, "lse"), _ptr(g, torch.float32, T, "g"), _ptr(logp, torch.float32, T, "logp"),
            _ptr(entropy, torch.float32, T, "entropy"), _ptr(w, torch.float32, R, "w"), C.c_float(grad_scale),
            _ptr(dH, dt, T * d, "dH"), _ptr(dW, torch.float32, V * d, "dW"), 1 if accumulate_dW else 0,
            workspace.data_ptr(), workspace.numel())
        _check(rc, "aero_grpo_loss_reg_bwd")
        return dH, dW

    def fwd_bwd_workspace_bytes(self, T, d, V, R, chunk_tokens):
        return self.lib.aero_fwd_bwd_workspace_bytes(T, d, V, R, chunk_tokens)

    def grpo_loss_fwd_bwd(self, cfg, H, W, y, old_logp, cs, adv, w, keep, out=None, grad_scale=1.0, dH=None, dW=None,
                          accumulate_dW=False, chunk_tokens=None, workspace=None, ref_logp=None, entropy=False):
        """aero_grpo_loss_fwd_bwd (aero_grpo_loss_kl_fwd_bwd when ref_logp is given, aero_grpo_loss_reg_fwd_bwd when
        the entropy term is asked for): forward and backward of stage (b) in one call (no recompute of the
        logits).  Returns (forward outputs dict, dH, dW)."""
        T, d = H.shape
        V = W.shape[0]
        R = cs.numel() - 1
        dt = torch.bfloat16 if cfg.dtype == AERO_BF16 else torch.float32
        o = out if out is not None else {}
        for name in ("logp", "lse", "g"):
            if name not in o:
                o[name] = torch.empty(max(T, 1), dtype=torch.float32, device=self.device)
        if "loss" not in o:
            o["loss"] = torch.zeros(1, dtype=torch.float32, device=self.device)
        if "metrics" not in o:
            o["metrics"] = torch.zeros(4, dtype=torch.float32, device=self.device)
        if dH is None:
            dH = torch.empty((max(T, 1), d), dtype=dt, device=self.device)[:T]
        if dW is None:
            dW = torch.empty((V, d), dtype=torch.float32, device=self.device)
        if workspace is None:
            if chunk_tokens is None:
                chunk_tokens = min(max(128, (T + 127) // 128 * 128), 2 * 148 * 128)
            workspace = self.workspace(self.fwd_bwd_workspace_bytes(T, d, V, R, chunk_tokens))
        head = (self.h, C.byref(cfg), T, d, V, R, _ptr(H, dt, T * d, "H"), _ptr(W, dt, V * d, "W"),
                _ptr(y, torch.int32, T, "y"), _ptr(old_logp, torch.float32, T, "old_logp"))
        tail = (_ptr(cs, torch.int64, R + 1, "cs"), _ptr(adv, torch.float32, R, "adv"), _ptr(w, torch.float32, R, "w"),
                _ptr(keep, torch.uint8, R, "keep"), _ptr(o["logp"]), _ptr(o["lse"]), _ptr(o["g"]), _ptr(o["loss"]),
                _ptr(o["metrics"]), C.c_float(grad_scale), _ptr(dH, dt, T * d, "dH"), _ptr(dW, torch.float32, V * d, "dW"),
                1 if accumulate_dW else 0, workspace.data_ptr(), workspace.numel())
        if entropy:
            if "entropy" not in o:
                o["entropy"] = torch.empty(max(T, 1), dtype=torch.float32, device=self.device)
            ref = _ptr(ref_logp, torch.float32, T, "ref_logp") if ref_logp is not None else None
            _check(self.lib.aero_grpo_loss_reg_fwd_bwd(*head, ref, *tail[:7], _ptr(o["entropy"]), *tail[7:]),
                   "aero_grpo_loss_reg_fwd_bwd")
        elif ref_logp is None:
            _check(self.lib.aero_grpo_loss_fwd_bwd(*head, *tail), "aero_grpo_loss_fwd_bwd")
        else:
            _check(self.lib.aero_grpo_loss_kl_fwd_bwd(*head, _ptr(ref_logp, torch.float32, T, "ref_logp"), *tail),
                   "aero_grpo_loss_kl_fwd_bwd")
        return o, dH, dW

    def grpo_loss_bwd(self, cfg, H, W, y, cs, keep, lse, g, grad_scale=1.0, dH=None, dW=None,
                      accumulate_dW=False, chunk_tokens=None, workspace=None, logp=None):
        T, d = H.shape
        V = W.shape[0]
        R = cs.numel() - 1
        dt = torch.bfloat16 if cfg.dtype == AERO_BF16 else torch.float32
        if dH is None:
            dH = torch.empty((max(T, 1), d), dtype=dt, device=self.device)[:T]
        if dW is None:
            dW = torch.empty((V, d), dtype=torch.float32, device=self.device)
        if workspace is None:
            if chunk_tokens is None:
                chunk_tokens = min(max(128, (T + 127) // 128 * 128), 2 * 148 * 128)
            workspace = self.workspace(self.bwd_workspace_bytes(T, d, V, R, chunk_tokens))
        rc = self.lib.aero_grpo_loss_bwd(
            self.h, C.byref(cfg), T, d, V, R, _ptr(H, dt, T * d, "H"), _ptr(W, dt, V * d, "W"),
            _ptr(y, torch.int32, T, "y"), _ptr(cs, torch.int64, R + 1, "cs"), _ptr(keep, torch.uint8, R, "keep"),
            _ptr(lse, torch.float32, T, "lse"), _ptr(g, torch.float32, T, "g"), _ptr(logp, torch.float32, T, "logp"),
            C.c_float(grad_scale),
            _ptr(dH, dt, T * d, "dH"), _ptr(dW, torch.float32, V * d, "dW"), 1 if accumulate_dW else 0,
            workspace.data_ptr(), workspace.numel())
        _check(rc, "aero_grpo_loss_bwd")
        return dH, dW

    # ---- allocation controller, simulated ----------------------------------------------------
    def allocate_sim(self, cfg, acfg, thr, out=None):
        """aero_allocate_sim: thr is a 32-bit integer CUDA tensor (bits read as unsigned) of per-prompt
        success thresholds; returns n_gen, c, n_train [P] int32 and counters [8] int64."""
        P = thr.numel()
        if thr.dtype not in (torch.int32, torch.uint32):
            raise AeroError("thr must be a 32-bit integer tensor (its bits are read as unsigned)")
        o = out if out is not None else {}
        for name in ("n_gen", "c", "n_train"):
            if name not in o:
                o[name] = torch.empty(max(P, 1), dtype=torch.int32, device=self.device)
        if "counters" not in o:
            o["counters"] = torch.zeros(8, dtype=torch.int64, device=self.device)
        ws = self.workspace(self.lib.aero_allocate_workspace_bytes(P))
        rc = self.lib.aero_allocate_sim(self.h, C.byref(cfg), C.byref(acfg), P, _ptr(thr, None, P, "thr"),
                                        _ptr(o["n_gen"]), _ptr(o["c"]), _ptr(o["n_train"]), _ptr(o["counters"]),
                                        ws.data_ptr(), ws.numel())
        _check(rc, "aero_allocate_sim")
        return o

    def enable_kernel_timing(self, on=True):
        _check(self.lib.aero_enable_kernel_timing(self.h, 1 if on else 0), "aero_enable_kernel_timing")

    def kernel_timing_ms(self):
        """(summed ms, launches) of the lm_head launches of grpo_loss_fwd_bwd since the last read-out."""
        ms, n = C.c_float(0), C.c_int(0)
        _check(self.lib.aero_kernel_timing_ms(self.h, C.byref(ms), C.byref(n)), "aero_kernel_timing_ms")
        return ms.value, n.value

    # ---- whole step from host buffers ---------------------------------------------------
    def launch_count(self) -> int:
        return int(self.lib.aero_launch_count(self.h))

    def step_workspace_bytes(self, P, R, T, d, V, chunk_tokens, dtype=AERO_BF16):
        return self.lib.aero_step_workspace_bytes(P, R, T, d, V, chunk_tokens, dtype)

    def grpo_step_host(self, cfg, go_h, reward_h, cs_h, key_h, alpha_h, beta_h, H_h, y_h, old_h, W, dH, dW,
                       workspace, accumulate_dW=False):
        """Host tensors (ideally pinned) in, device W/dH/dW, returns (loss, counters, metrics) host tensors."""
        P, R = go_h.numel() - 1, reward_h.numel()
        T, d = H_h.shape
        V = W.shape[0]

        def hp(t):
            if t is None:
                return None
            if t.is_cuda or not t.is_contiguous():
                raise AeroError("host inputs must be contiguous CPU tensors")
            return t.data_ptr()

        loss = torch.zeros(1, dtype=torch.float32)
        counters = torch.zeros(8, dtype=torch.int64)
        metrics = torch.zeros(8, dtype=torch.float32)
        rc = self.lib.aero_grpo_step_host(
            self.h, C.byref(cfg), P, R, T, d, V, hp(go_h), hp(reward_h), hp(cs_h), hp(key_h), hp(alpha_h), hp(beta_h),
            hp(H_h), hp(y_h), hp(old_h), _ptr(W), _ptr(dH), _ptr(dW, torch.float32), 1 if accumulate_dW else 0,
            loss.data_ptr(), counters.data_ptr(), metrics.data_ptr(), workspace.data_ptr(), workspace.numel())
        _check(rc, "aero_grpo_step_host")
        return loss, counters, metrics
