"""ctypes binding of libpbt_b200.so: argument marshalling only.

Every step of the hot path runs inside the library's CUDA kernels.  PyTorch is
used here for device memory (the workspace and the data pools) and for the
stream; nothing in this module computes any part of the method, and there is no
fallback: if the shared library or a CUDA device is missing, calls raise.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Dict, Optional

import numpy as np

PBT_MAX_LAYERS = 8
PBT_MAX_NH = 8
PBT_N_SCALARS = 4
PBT_HISTORY = 10

_DTYPE = {"fp64_toy": 0, "fp32": 1, "bf16_fp32master": 2}
_MODEL = {"toy_quadratic": 0, "mlp": 1, "gan_pair": 2}
_LOSS = {"toy": 0, "mse": 1, "ce_hard": 2, "ce_soft": 3, "gan_logistic": 4, "wgan_gp": 5}
_OPT = {"sgd_plain": 0, "sgdm": 1, "adam": 2, "rmsprop": 3}

STATUS = {0: "PBT_OK", 1: "PBT_ERR_INVALID_ARG", 2: "PBT_ERR_UNSUPPORTED", 3: "PBT_ERR_WORKSPACE",
          4: "PBT_ERR_CUDA", 5: "PBT_ERR_TIMEOUT", 6: "PBT_ERR_STATE"}


class PbtSpec(C.Structure):
    _fields_ = [
        ("n_members", C.c_int32), ("dtype", C.c_int32), ("model", C.c_int32), ("loss", C.c_int32),
        ("optimizer", C.c_int32), ("n_layers", C.c_int32 * 2),
        ("widths", (C.c_int32 * (PBT_MAX_LAYERS + 1)) * 2),
        ("batch", C.c_int32), ("eval_batch", C.c_int32), ("pool_rows", C.c_int32),
        ("gan_d_steps", C.c_int32), ("nh", C.c_int32),
        ("slot_lr", C.c_int32), ("slot_lr_d", C.c_int32), ("slot_momentum", C.c_int32),
        ("slot_beta1", C.c_int32), ("slot_wd", C.c_int32),
        ("perturb_mask", C.c_uint32), ("flags", C.c_uint32),
        ("trunc_num", C.c_int32), ("trunc_den", C.c_int32), ("keep_grad", C.c_int32), ("fuse_adam", C.c_int32), ("programmatic_launches", C.c_int32), ("backward_streams", C.c_int32), ("member_base", C.c_int32), ("n_global", C.c_int32), ("exploit_rule", C.c_int32),
        ("explore_rule", C.c_int32), ("prior_kind", C.c_int32 * PBT_MAX_NH),
        ("const_lr", C.c_double), ("const_momentum", C.c_double), ("const_beta1", C.c_double),
        ("const_beta2", C.c_double), ("const_eps", C.c_double), ("const_wd", C.c_double),
        ("toy_eta", C.c_double), ("toy_theta0", C.c_double * PBT_MAX_NH),
        ("factor_lo", C.c_double), ("factor_hi", C.c_double),
        ("clamp_lo", C.c_double * PBT_MAX_NH), ("clamp_hi", C.c_double * PBT_MAX_NH),
        ("ttest_alpha", C.c_double), ("resample_prob", C.c_double),
        ("prior_lo", C.c_double * PBT_MAX_NH), ("prior_hi", C.c_double * PBT_MAX_NH),
        ("gp_lambda", C.c_double),
    ]


class PbtData(C.Structure):
    _fields_ = [("x_pool", C.c_void_p), ("y_pool", C.c_void_p), ("z_pool", C.c_void_p),
                ("x_eval", C.c_void_p), ("y_eval", C.c_void_p)]


class PbtStateView(C.Structure):
    _fields_ = [("w", C.c_void_p), ("opt1", C.c_void_p), ("opt2", C.c_void_p), ("grad", C.c_void_p),
                ("scalars", C.POINTER(C.c_double)), ("hparams", C.POINTER(C.c_double)),
                ("fitness", C.POINTER(C.c_double)), ("step", C.POINTER(C.c_int64)),
                ("round", C.POINTER(C.c_int64))]


class PbtGemmDesc(C.Structure):
    _fields_ = [("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32), ("batch", C.c_int32),
                ("in_bf16", C.c_int32), ("out_bf16", C.c_int32), ("a_mn", C.c_int32), ("b_mn", C.c_int32),
                ("relu", C.c_int32), ("engine", C.c_int32),
                ("A", C.c_void_p), ("lda", C.c_int64), ("strideA", C.c_int64),
                ("B", C.c_void_p), ("ldb", C.c_int64), ("strideB", C.c_int64),
                ("C", C.c_void_p), ("ldc", C.c_int64), ("strideC", C.c_int64),
                ("bias", C.c_void_p), ("strideBias", C.c_int64),
                ("mask", C.c_void_p), ("ldmask", C.c_int64), ("strideMask", C.c_int64),
                ("status_device", C.c_void_p)]


EXPORTS = [
    "pbt_query_workspace", "pbt_param_count", "pbt_create", "pbt_destroy", "pbt_step", "pbt_step_subset", "pbt_eval",
    "pbt_exploit_explore", "pbt_exploit_explore_ready", "pbt_exploit_explore_global", "pbt_set_global_history",
    "pbt_copy_members_level",
    "pbt_member_slabs", "pbt_get_state", "pbt_set_state", "pbt_get_fitness", "pbt_set_fitness",
    "pbt_get_history", "pbt_set_history",
    "pbt_get_hparams", "pbt_set_hparams", "pbt_get_copy_map", "pbt_get_best", "pbt_get_last_loss",
    "pbt_set_batch", "pbt_step_host", "pbt_prefetch_host_batch", "pbt_step_prefetched", "pbt_get_launch_count", "pbt_profile_begin", "pbt_profile_end", "pbt_profile_get",
    "pbt_grouped_gemm", "pbt_selftest_bounded_wait", "pbt_energy_fitness_static", "pbt_last_error",
]

_LIB = None


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libpbt_b200.so")


def load_library() -> C.CDLL:
    """dlopen the CUDA library; raises if it has not been built (no fallback exists)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run paper_1711_09846_b200/build.py (nvcc, sm_100a); "
                           "there is no CPU or PyTorch fallback")
    lib = C.CDLL(path)
    vp = C.c_void_p
    lib.pbt_query_workspace.argtypes = [C.POINTER(PbtSpec), C.POINTER(C.c_size_t)]
    lib.pbt_param_count.argtypes = [C.POINTER(PbtSpec), C.POINTER(C.c_int64)]
    lib.pbt_create.argtypes = [C.POINTER(vp), C.POINTER(PbtSpec), C.POINTER(C.c_double), C.c_uint64,
                               C.POINTER(PbtData), vp, C.c_size_t, vp]
    lib.pbt_destroy.argtypes = [vp]
    lib.pbt_step.argtypes = [vp, C.c_int]
    lib.pbt_step_subset.argtypes = [vp, C.POINTER(C.c_uint8), C.c_int]
    lib.pbt_eval.argtypes = [vp]
    lib.pbt_exploit_explore.argtypes = [vp]
    lib.pbt_exploit_explore_ready.argtypes = [vp, C.POINTER(C.c_uint8)]
    lib.pbt_exploit_explore_global.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_uint8),
                                               C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.pbt_set_global_history.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int32)]
    lib.pbt_copy_members_level.argtypes = [vp, C.c_int]
    lib.pbt_member_slabs.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(C.c_size_t), C.POINTER(C.c_int32)]
    lib.pbt_get_state.argtypes = [vp, C.c_int, C.POINTER(PbtStateView)]
    lib.pbt_set_state.argtypes = [vp, C.c_int, C.POINTER(PbtStateView)]
    lib.pbt_get_fitness.argtypes = [vp, C.POINTER(C.c_double)]
    lib.pbt_set_fitness.argtypes = [vp, C.POINTER(C.c_double)]
    lib.pbt_get_hparams.argtypes = [vp, C.POINTER(C.c_double)]
    lib.pbt_set_hparams.argtypes = [vp, C.POINTER(C.c_double)]
    lib.pbt_get_copy_map.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.pbt_get_best.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.pbt_get_last_loss.argtypes = [vp, C.POINTER(C.c_double)]
    lib.pbt_set_batch.argtypes = [vp, vp, vp]
    lib.pbt_step_host.argtypes = [vp, vp, vp, C.POINTER(C.c_double)]
    lib.pbt_prefetch_host_batch.argtypes = [vp, vp, vp]
    lib.pbt_step_prefetched.argtypes = [vp, C.POINTER(C.c_double)]
    lib.pbt_get_launch_count.argtypes = [vp, C.POINTER(C.c_int64)]
    lib.pbt_profile_begin.argtypes = [vp]
    lib.pbt_profile_end.argtypes = [vp]
    lib.pbt_profile_get.argtypes = [vp, C.c_char_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.pbt_grouped_gemm.argtypes = [C.POINTER(PbtGemmDesc), vp]
    lib.pbt_energy_fitness_static.argtypes = [vp, C.c_int, C.c_int, vp, vp]
    lib.pbt_selftest_bounded_wait.argtypes = [vp, C.c_int, vp]
    lib.pbt_last_error.argtypes = [vp]
    lib.pbt_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name != "pbt_last_error":
            getattr(lib, name).restype = C.c_int
    _LIB = lib
    return lib


class PbtError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{STATUS.get(code, code)}: {msg}")
        self.code = code


def spec_from_config(cfg, keep_grad: bool = False, fuse_adam: bool = True, programmatic_launches: bool = False,
                     backward_streams: int = 0) -> PbtSpec:
    """Translate a declarative population description (see workloads.configs.PBTConfig) into pbt_spec."""
    s = PbtSpec()
    s.n_members = cfg.n_members
    s.dtype = _DTYPE[cfg.dtype]
    s.model = _MODEL[cfg.model]
    s.loss = _LOSS[cfg.loss]
    s.optimizer = _OPT[cfg.optimizer]
    if cfg.model != "toy_quadratic":
        for k, ws in enumerate(cfg.widths):
            s.n_layers[k] = len(ws) - 1
            for l, w in enumerate(ws):
                s.widths[k][l] = w
    s.batch, s.eval_batch, s.pool_rows = cfg.batch, cfg.eval_batch, cfg.pool_rows
    s.gan_d_steps = cfg.gan_d_steps
    s.nh = cfg.nh
    s.slot_lr = cfg.slot("lr")
    s.slot_lr_d = cfg.slot("lr_d")
    s.slot_momentum = cfg.slot("momentum")
    s.slot_beta1 = cfg.slot("beta1")
    s.slot_wd = cfg.slot("wd")
    mask = 0
    for k, on in enumerate(cfg.perturb):
        mask |= (1 << k) if on else 0
    s.perturb_mask = mask
    s.flags = cfg.flags
    s.trunc_num, s.trunc_den = cfg.trunc_num, cfg.trunc_den
    s.keep_grad = 1 if keep_grad else 0
    s.programmatic_launches = 1 if programmatic_launches else 0
    s.backward_streams = int(backward_streams)
    s.exploit_rule = {"truncation": 0, "tournament": 1, "ttest": 2}[getattr(cfg, "exploit", "truncation")]
    s.explore_rule = {"perturb": 0, "resample": 1}[getattr(cfg, "explore", "perturb")]
    s.ttest_alpha = getattr(cfg, "ttest_alpha", 0.05)
    s.resample_prob = getattr(cfg, "resample_prob", 0.25)
    for k, (kind, lo, hi) in enumerate(cfg.priors[:cfg.nh]):
        s.prior_kind[k] = {"fixed": 0, "u": 1, "logu": 2}[kind]
        s.prior_lo[k], s.prior_hi[k] = lo, hi
    s.fuse_adam = 1 if fuse_adam else 0
    s.gp_lambda = getattr(cfg, "gp_lambda", 10.0)
    s.const_lr = 0.0
    s.const_momentum = cfg.momentum
    s.const_beta1, s.const_beta2, s.const_eps, s.const_wd = cfg.beta1, cfg.beta2, cfg.eps, cfg.weight_decay
    s.toy_eta = cfg.toy_eta
    for k, v in enumerate(cfg.toy_theta0):
        s.toy_theta0[k] = v
    s.factor_lo, s.factor_hi = cfg.factor_lo, cfg.factor_hi
    for k in range(PBT_MAX_NH):
        s.clamp_lo[k] = cfg.clamp_lo[k] if k < len(cfg.clamp_lo) else -math.inf
        s.clamp_hi[k] = cfg.clamp_hi[k] if k < len(cfg.clamp_hi) else math.inf
    return s


def param_count(cfg) -> int:
    lib = load_library()
    n = C.c_int64(0)
    spec = spec_from_config(cfg)
    rc = lib.pbt_param_count(C.byref(spec), C.byref(n))
    if rc:
        raise PbtError(rc, lib.pbt_last_error(None).decode())
    return n.value


def grouped_gemm(A, B, C_out, a_mn=False, b_mn=False, bias=None, relu=False, mask=None, engine=0, status=None,
                 stream=None, shared_a=False, shared_b=False):
    """C_b = epilogue(A_b B_b^T) for every b; torch CUDA tensors, marshalling only (see pbt_grouped_gemm).

    A: [batch, M, K] (or [batch, K, M] when a_mn); B: [batch, N, K] (or [batch, K, N] when b_mn);
    C_out: [batch, M, N] float32 or bfloat16, written in place.  bias: [batch, N] float32;
    mask: [batch, M, N] in the operand dtype.  status: >= 8 zeroed int32 on the device."""
    import torch
    lib = load_library()
    d = PbtGemmDesc()
    batch, M, N = C_out.shape
    K = A.shape[1] if a_mn else A.shape[2]
    d.M, d.N, d.K, d.batch = M, N, K, batch
    d.in_bf16 = 1 if A.dtype == torch.bfloat16 else 0
    d.out_bf16 = 1 if C_out.dtype == torch.bfloat16 else 0
    d.a_mn, d.b_mn, d.relu, d.engine = int(a_mn), int(b_mn), int(relu), int(engine)
    d.A, d.lda, d.strideA = A.data_ptr(), A.stride(1), 0 if shared_a else A.stride(0)
    d.B, d.ldb, d.strideB = B.data_ptr(), B.stride(1), 0 if shared_b else B.stride(0)
    d.C, d.ldc, d.strideC = C_out.data_ptr(), C_out.stride(1), C_out.stride(0)
    if bias is not None:
        d.bias, d.strideBias = bias.data_ptr(), bias.stride(0)
    if mask is not None:
        d.mask, d.ldmask, d.strideMask = mask.data_ptr(), mask.stride(1), mask.stride(0)
    if status is not None:
        d.status_device = status.data_ptr()
    rc = lib.pbt_grouped_gemm(C.byref(d), C.c_void_p(stream.cuda_stream if stream is not None else None))
    if rc:
        raise PbtError(rc, lib.pbt_last_error(None).decode())


def selftest_bounded_wait(status, polls: int = 2000, stream=None) -> None:
    """Run the kernels' bounded barrier wait on a barrier nothing signals (see pbt_selftest_bounded_wait);
    status: >= 8 zeroed int32 on the device, status[4] becomes PBT_ERR_TIMEOUT."""
    lib = load_library()
    rc = lib.pbt_selftest_bounded_wait(C.c_void_p(status.data_ptr()), int(polls),
                                       C.c_void_p(stream.cuda_stream if stream is not None else None))
    if rc:
        raise PbtError(rc, lib.pbt_last_error(None).decode())


def energy_fitness_static(x_dev, fitness_out_dev, stream=None) -> None:
    """Score point sets without any device allocation (see pbt_energy_fitness_static in pbt.h).

    x_dev: CUDA float32 tensor [n_members, n, 2]; fitness_out_dev: CUDA float32 tensor [n_members],
    written in place.  Only enqueues work on `stream` (a torch stream, or None for the default one).
    Meant for hosts that may not allocate: the reduction's scratch is a fixed array in the library."""
    lib = load_library()
    assert x_dev.is_cuda and x_dev.is_contiguous() and x_dev.dim() == 3 and x_dev.shape[2] == 2
    assert fitness_out_dev.is_cuda and fitness_out_dev.is_contiguous() and fitness_out_dev.numel() == x_dev.shape[0]
    rc = lib.pbt_energy_fitness_static(C.c_void_p(x_dev.data_ptr()), int(x_dev.shape[1]), int(x_dev.shape[0]),
                                       C.c_void_p(fitness_out_dev.data_ptr()),
                                       C.c_void_p(stream.cuda_stream if stream is not None else None))
    if rc:
        raise PbtError(rc, lib.pbt_last_error(None).decode())


class Population:
    """One population living on one GPU.  Thin wrapper over the pbt_* calls."""

    def __init__(self, cfg, inputs, seed: Optional[int] = None, device: str = "cuda:0", keep_grad: bool = False,
                 fuse_adam: bool = True, guard_bytes: int = 0, programmatic_launches: bool = False,
                 member_base: int = 0, n_global: int = 0, backward_streams: int = 0):
        """cfg.n_members members on `device`.  member_base / n_global: this population is the shard
        [member_base, member_base + cfg.n_members) of a population of n_global members (see sharding.py);
        inputs.init_hparams then holds the rows of the whole population."""
        import torch
        self._torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: this library has no CPU path")
        self.cfg = cfg
        self.device = torch.device(device)
        self.seed = int(cfg.seed if seed is None else seed)
        self.spec = spec_from_config(cfg, keep_grad, fuse_adam, programmatic_launches, backward_streams)
        self.member_base, self.n_global = int(member_base), int(n_global)
        self.spec.member_base, self.spec.n_global = self.member_base, self.n_global
        self.N, self.nh = cfg.n_members, cfg.nh
        self.toy = cfg.model == "toy_quadratic"
        torch.cuda.set_device(self.device)
        self.stream = torch.cuda.Stream(device=self.device)
        self._keep = []
        data = PbtData()
        if not self.toy:
            op_dtype = torch.bfloat16 if cfg.dtype == "bf16_fp32master" else torch.float32

            def dev(a, dtype):
                if a is None:
                    return None
                t = torch.from_numpy(np.ascontiguousarray(a)).to(self.device).to(dtype).contiguous()
                self._keep.append(t)
                return t

            ydt = {"mse": torch.float32, "ce_hard": torch.int32, "ce_soft": op_dtype}.get(cfg.loss, op_dtype)
            self.x_pool = dev(inputs.x_pool, op_dtype)
            self.y_pool = dev(inputs.y_pool, ydt)
            self.z_pool = dev(inputs.z_pool, op_dtype)
            self.x_eval = dev(inputs.x_eval, op_dtype)
            self.y_eval = dev(inputs.y_eval, ydt)
            for name in ("x_pool", "y_pool", "z_pool", "x_eval", "y_eval"):
                t = getattr(self, name)
                setattr(data, name, t.data_ptr() if t is not None else None)
        nbytes = C.c_size_t(0)
        self._check(self.lib.pbt_query_workspace(C.byref(self.spec), C.byref(nbytes)), None)
        self.workspace_bytes = nbytes.value
        # optional guard bands on both sides of the workspace (a debugging aid: guards_intact() tells whether any
        # kernel wrote outside the memory the library was given)
        self.guard_bytes = (int(guard_bytes) + 255) // 256 * 256
        self.workspace = torch.empty(nbytes.value + 256 + 2 * self.guard_bytes, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + self.guard_bytes + 255) // 256 * 256
        self._ws_off = base - self.workspace.data_ptr()
        if self.guard_bytes:
            self.workspace[:self._ws_off].fill_(0xA5)
            self.workspace[self._ws_off + nbytes.value:].fill_(0xA5)
        h0 = np.ascontiguousarray(inputs.init_hparams, dtype=np.float64)
        if self.n_global:
            assert h0.shape == (self.n_global, self.nh)
            h0 = np.ascontiguousarray(h0[self.member_base:self.member_base + self.N])
        assert h0.shape == (self.N, self.nh)
        self.handle = C.c_void_p(None)
        torch.cuda.synchronize(self.device)
        rc = self.lib.pbt_create(C.byref(self.handle), C.byref(self.spec),
                                 h0.ctypes.data_as(C.POINTER(C.c_double)), C.c_uint64(self.seed),
                                 C.byref(data), C.c_void_p(base), C.c_size_t(nbytes.value),
                                 C.c_void_p(self.stream.cuda_stream))
        self._check(rc, None)
        n = C.c_int64(0)
        self._check(self.lib.pbt_param_count(C.byref(self.spec), C.byref(n)), None)
        self.n_params = n.value

    # ------------------------------------------------------------------
    def _check(self, rc, handle=True):
        if rc != 0:
            h = self.handle if (handle and getattr(self, "handle", None)) else None
            raise PbtError(rc, self.lib.pbt_last_error(h).decode())

    def close(self):
        if getattr(self, "handle", None):
            self.synchronize()
            self.lib.pbt_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def synchronize(self):
        self.stream.synchronize()

    def guards_intact(self) -> bool:
        """True if the guard bands around the workspace (guard_bytes at construction) still hold their fill."""
        assert self.guard_bytes > 0, "construct the population with guard_bytes > 0"
        self.synchronize()
        lo = self.workspace[:self._ws_off]
        hi = self.workspace[self._ws_off + self.workspace_bytes:]
        return bool((lo == 0xA5).all().item()) and bool((hi == 0xA5).all().item())

    # ----- the hot path ---------------------------------------------------
    def step(self, k: int = 1):
        self._check(self.lib.pbt_step(self.handle, int(k)))

    def step_subset(self, active, k: int = 1):
        """k steps for the members whose entry of `active` (bools, one per member) is set; the others sit out."""
        mask = np.ascontiguousarray(np.asarray(active, dtype=bool).astype(np.uint8))
        assert mask.shape == (self.cfg.n_members,)
        self._check(self.lib.pbt_step_subset(self.handle, mask.ctypes.data_as(C.POINTER(C.c_uint8)), int(k)))

    def eval(self):
        self._check(self.lib.pbt_eval(self.handle))

    def exploit_explore(self, ready=None):
        """One ready point; `ready` (bools, one per member; None = everybody) says which members may exploit now."""
        if ready is None:
            self._check(self.lib.pbt_exploit_explore(self.handle))
            return
        mask = np.ascontiguousarray(np.asarray(ready, dtype=bool).astype(np.uint8))
        assert mask.shape == (self.cfg.n_members,)
        self._check(self.lib.pbt_exploit_explore_ready(self.handle, mask.ctypes.data_as(C.POINTER(C.c_uint8))))

    # ----- sharded populations (see sharding.py) ---------------------------
    def exploit_explore_global(self, fitness_global, hparams_global, ready=None):
        """Selection and explore for the WHOLE population on this shard's device (every shard gets the same answer);
        returns (src, level, n_levels, fitness_after, hparams_after) in indices of the whole population and
        applies the rows of this shard's members to its own records.  Moves no weights."""
        G = self.n_global
        f = np.ascontiguousarray(fitness_global, dtype=np.float64).copy()
        h = np.ascontiguousarray(hparams_global, dtype=np.float64).copy()
        assert f.shape == (G,) and h.shape == (G, self.nh)
        src, level = np.zeros(G, dtype=np.int32), np.zeros(G, dtype=np.int32)
        n_levels = C.c_int32(0)
        mask = None
        if ready is not None:
            mask = np.ascontiguousarray(np.asarray(ready, dtype=bool).astype(np.uint8))
            assert mask.shape == (G,)
        self._check(self.lib.pbt_exploit_explore_global(
            self.handle, f.ctypes.data_as(C.POINTER(C.c_double)), h.ctypes.data_as(C.POINTER(C.c_double)),
            mask.ctypes.data_as(C.POINTER(C.c_uint8)) if mask is not None else None,
            src.ctypes.data_as(C.POINTER(C.c_int32)), level.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(n_levels)))
        return src, level, n_levels.value, f, h

    def set_global_history(self, hist_global, count_global):
        """The whole population's score histories for the next exploit_explore_global (t-test selection)."""
        h = np.ascontiguousarray(hist_global, dtype=np.float64)
        c = np.ascontiguousarray(count_global, dtype=np.int32)
        assert h.shape == (self.n_global, PBT_HISTORY) and c.shape == (self.n_global,)
        self._check(self.lib.pbt_set_global_history(self.handle, h.ctypes.data_as(C.POINTER(C.c_double)),
                                                    c.ctypes.data_as(C.POINTER(C.c_int32))))

    def copy_members_level(self, level: int):
        self._check(self.lib.pbt_copy_members_level(self.handle, int(level)))

    def member_slabs(self, m: int):
        """The arrays of local member m's copied record as uint8 views of the workspace (device memory, no copy)."""
        ptrs, sizes, n = (C.c_void_p * 5)(), (C.c_size_t * 5)(), C.c_int32(0)
        self._check(self.lib.pbt_member_slabs(self.handle, int(m), ptrs, sizes, C.byref(n)))
        base = self.workspace.data_ptr()
        return [self.workspace[ptrs[i] - base:ptrs[i] - base + sizes[i]] for i in range(n.value)]

    # ----- state access ---------------------------------------------------
    def get_state(self, m: int) -> Dict[str, np.ndarray]:
        dt = np.float64 if self.toy else np.float32
        P = self.n_params
        out = {k: np.zeros(P, dtype=dt) for k in (("w",) if self.toy else ("w", "opt1", "opt2", "grad"))}
        sc = np.zeros(PBT_N_SCALARS, dtype=np.float64)
        hp = np.zeros(max(self.nh, 1), dtype=np.float64)
        fit = C.c_double(0)
        step, rnd = C.c_int64(0), C.c_int64(0)
        v = PbtStateView()
        for k, a in out.items():
            setattr(v, k, a.ctypes.data)
        v.scalars = sc.ctypes.data_as(C.POINTER(C.c_double))
        v.hparams = hp.ctypes.data_as(C.POINTER(C.c_double))
        v.fitness = C.pointer(fit)
        v.step = C.pointer(step)
        v.round = C.pointer(rnd)
        self._check(self.lib.pbt_get_state(self.handle, int(m), C.byref(v)))
        out.update(scalars=sc, hparams=hp[:self.nh], fitness=fit.value, step=step.value, round=rnd.value)
        return out

    def step_count(self, m: int = 0) -> int:
        """Member m's own step count t (Algorithm 1's t); reads one counter, not the member's record."""
        step = C.c_int64(0)
        v = PbtStateView()
        v.step = C.pointer(step)
        self._check(self.lib.pbt_get_state(self.handle, int(m), C.byref(v)))
        return step.value

    def set_state(self, m: int, w=None, opt1=None, opt2=None, scalars=None, hparams=None, fitness=None,
                  step=None, round=None):
        dt = np.float64 if self.toy else np.float32
        keep = []
        v = PbtStateView()
        for name, a in (("w", w), ("opt1", opt1), ("opt2", opt2)):
            if a is not None:
                a = np.ascontiguousarray(a, dtype=dt)
                assert a.size == self.n_params
                keep.append(a)
                setattr(v, name, a.ctypes.data)
        if scalars is not None:
            a = np.ascontiguousarray(scalars, dtype=np.float64)
            keep.append(a)
            v.scalars = a.ctypes.data_as(C.POINTER(C.c_double))
        if hparams is not None:
            a = np.ascontiguousarray(hparams, dtype=np.float64)
            keep.append(a)
            v.hparams = a.ctypes.data_as(C.POINTER(C.c_double))
        if fitness is not None:
            f = C.c_double(float(fitness))
            keep.append(f)
            v.fitness = C.pointer(f)
        if step is not None:
            s_ = C.c_int64(int(step))
            keep.append(s_)
            v.step = C.pointer(s_)
        if round is not None:
            r_ = C.c_int64(int(round))
            keep.append(r_)
            v.round = C.pointer(r_)
        self._check(self.lib.pbt_set_state(self.handle, int(m), C.byref(v)))

    def fitness(self) -> np.ndarray:
        f = np.zeros(self.N, dtype=np.float64)
        self._check(self.lib.pbt_get_fitness(self.handle, f.ctypes.data_as(C.POINTER(C.c_double))))
        return f

    def history(self):
        """(scores [N][PBT_HISTORY] oldest first, counts [N]) used by t-test selection."""
        h = np.zeros((self.N, PBT_HISTORY), dtype=np.float64)
        c = np.zeros(self.N, dtype=np.int32)
        self._check(self.lib.pbt_get_history(self.handle, h.ctypes.data_as(C.POINTER(C.c_double)),
                                             c.ctypes.data_as(C.POINTER(C.c_int32))))
        return h, c

    def set_history(self, h, c):
        h = np.ascontiguousarray(h, dtype=np.float64)
        c = np.ascontiguousarray(c, dtype=np.int32)
        assert h.shape == (self.N, PBT_HISTORY) and c.shape == (self.N,)
        self._check(self.lib.pbt_set_history(self.handle, h.ctypes.data_as(C.POINTER(C.c_double)),
                                             c.ctypes.data_as(C.POINTER(C.c_int32))))

    def set_fitness(self, f):
        f = np.ascontiguousarray(f, dtype=np.float64)
        assert f.shape == (self.N,)
        self._check(self.lib.pbt_set_fitness(self.handle, f.ctypes.data_as(C.POINTER(C.c_double))))

    def hparams(self) -> np.ndarray:
        h = np.zeros((self.N, self.nh), dtype=np.float64)
        self._check(self.lib.pbt_get_hparams(self.handle, h.ctypes.data_as(C.POINTER(C.c_double))))
        return h

    def set_hparams(self, h):
        h = np.ascontiguousarray(h, dtype=np.float64)
        assert h.shape == (self.N, self.nh)
        self._check(self.lib.pbt_set_hparams(self.handle, h.ctypes.data_as(C.POINTER(C.c_double))))

    def copy_map(self) -> np.ndarray:
        s = np.zeros(self.N, dtype=np.int32)
        self._check(self.lib.pbt_get_copy_map(self.handle, s.ctypes.data_as(C.POINTER(C.c_int32))))
        return s

    def best(self) -> int:
        b = C.c_int32(0)
        self._check(self.lib.pbt_get_best(self.handle, C.byref(b)))
        return b.value

    def last_loss(self) -> np.ndarray:
        l = np.zeros((self.N, 2), dtype=np.float64)
        self._check(self.lib.pbt_get_last_loss(self.handle, l.ctypes.data_as(C.POINTER(C.c_double))))
        return l

    def set_batch(self, x_dev, y_dev):
        """x_dev [N, batch, in], y_dev matching targets: device tensors in the pools' dtypes."""
        assert x_dev.is_cuda and y_dev.is_cuda and x_dev.is_contiguous() and y_dev.is_contiguous()
        self._check(self.lib.pbt_set_batch(self.handle, C.c_void_p(x_dev.data_ptr()), C.c_void_p(y_dev.data_ptr())))

    def step_host(self, x_host, y_host, loss_out: Optional[np.ndarray] = None):
        """One step on rows held in host memory (torch CPU tensors, ideally pinned); returns the losses."""
        if loss_out is None:
            loss_out = np.zeros((self.N, 2), dtype=np.float64)
        self._check(self.lib.pbt_step_host(self.handle, C.c_void_p(x_host.data_ptr()), C.c_void_p(y_host.data_ptr()),
                                           loss_out.ctypes.data_as(C.POINTER(C.c_double))))
        return loss_out

    def prefetch_host_batch(self, x_host, y_host):
        """Start uploading the next step's rows (pinned torch CPU tensors) while the current step runs."""
        self._check(self.lib.pbt_prefetch_host_batch(self.handle, C.c_void_p(x_host.data_ptr()), C.c_void_p(y_host.data_ptr())))

    def step_prefetched(self, loss_out: Optional[np.ndarray] = None, wait: bool = True):
        """One step on the prefetched rows.  wait=False only enqueues (read the losses later with last_loss())."""
        if not wait:
            self._check(self.lib.pbt_step_prefetched(self.handle, None))
            return None
        if loss_out is None:
            loss_out = np.zeros((self.N, 2), dtype=np.float64)
        self._check(self.lib.pbt_step_prefetched(self.handle, loss_out.ctypes.data_as(C.POINTER(C.c_double))))
        return loss_out

    def launch_count(self) -> int:
        n = C.c_int64(0)
        self._check(self.lib.pbt_get_launch_count(self.handle, C.byref(n)))
        return n.value

    def profile_begin(self):
        self._check(self.lib.pbt_profile_begin(self.handle))

    def profile_end(self) -> Dict[str, Dict[str, float]]:
        self._check(self.lib.pbt_profile_end(self.handle))
        out = {}
        for cls in ("gemm", "wgrad_adam", "optimizer", "loss", "copy", "select", "other"):
            ms, n = C.c_double(0), C.c_int64(0)
            self._check(self.lib.pbt_profile_get(self.handle, cls.encode(), C.byref(ms), C.byref(n)))
            out[cls] = {"ms": ms.value, "launches": n.value}
        return out

    # ----- checkpoint / resume (Appendix A.1: members checkpoint themselves; here the whole population record) -----
    def state_dict(self) -> Dict[str, np.ndarray]:
        """The population record (theta, h, p, t) of every member plus optimiser state, score histories and the
        ready-point counter, as host arrays: enough to continue a run bit for bit with load_state_dict."""
        n = self.cfg.n_members
        members = [self.get_state(m) for m in range(n)]
        out = {"step": np.int64(members[0]["step"]), "round": np.int64(members[0]["round"]),
               "hparams": self.hparams(), "fitness": self.fitness(),
               "scalars": np.stack([s["scalars"] for s in members]),
               "w": np.stack([s["w"] for s in members])}
        if not self.toy:
            out["opt1"] = np.stack([s["opt1"] for s in members])
            out["opt2"] = np.stack([s["opt2"] for s in members])
        hist, count = self.history()
        out["history"], out["history_count"] = hist, count
        return out

    def load_state_dict(self, sd) -> None:
        n = self.cfg.n_members
        assert sd["w"].shape[0] == n and sd["hparams"].shape == (n, self.nh)
        for m in range(n):
            self.set_state(m, w=sd["w"][m], opt1=None if self.toy else sd["opt1"][m],
                           opt2=None if self.toy else sd["opt2"][m], scalars=sd["scalars"][m],
                           hparams=sd["hparams"][m], fitness=float(sd["fitness"][m]),
                           step=int(sd["step"]), round=int(sd["round"]))
        self.set_history(np.asarray(sd["history"], dtype=np.float64), np.asarray(sd["history_count"], dtype=np.int32))

    def save(self, path: str) -> None:
        np.savez(path, **self.state_dict())

    def load(self, path: str) -> None:
        with np.load(path) as z:
            self.load_state_dict({k: z[k] for k in z.files})

    # ----- Algorithm 1 in partial synchrony ---------------------------------
    def _ready_point(self, step, ready, log):
        """eval, exploit / explore and, if asked, one record of the ready point (Section 4.4's analyses are made
        from such records: score and hyperparameter traces, who copied whom)."""
        self.eval()
        if log is None:
            self.exploit_explore(ready)
            return
        rec = {"step": step, "ready": None if ready is None else [bool(r) for r in ready],
               "fitness": self.fitness(), "hparams_before": self.hparams()}
        self.exploit_explore(ready)
        rec["src"] = self.copy_map()
        rec["hparams_after"] = self.hparams()
        log.append(rec)

    @staticmethod
    def ancestors(log, n_members):
        """Initial member each current member descends from, following the copy maps of a ready-point log."""
        anc = list(range(n_members))
        for rec in log:
            anc = [anc[int(d)] for d in rec["src"]]
        return anc

    def run(self, total_steps: Optional[int] = None, log=None) -> int:
        """Algorithm 1 in partial synchrony: steps, and a ready point whenever `ready` holds.  `total_steps` is the
        ABSOLUTE step count to reach (default: the configuration's): the schedule is taken from the population's own
        step counter, so a population restored from a checkpoint (Appendix A.1) in the middle of an interval has its
        ready points at the same steps as the run that was never interrupted.  `log`: a list (or a bounded
        collections.deque) that receives one record per ready point; each record costs four small device-to-host
        reads."""
        cfg = self.cfg
        total = cfg.total_steps if total_steps is None else total_steps
        done = self.step_count(0)
        offsets = tuple(getattr(cfg, "ready_offsets", ())) or (0,) * cfg.n_members
        iv = cfg.ready_interval
        while done < total:
            # member m is ready when step - offsets[m] is a positive multiple of the interval (Algorithm 1's `ready`,
            # member by member; all offsets zero = everybody together): run to the next step at which anybody is
            nxt = min(o + iv * ((done - o) // iv + 1) if done >= o else o + iv for o in offsets)
            k = min(nxt, total) - done
            self.step(k)
            done += k
            ready = [(done - o) > 0 and (done - o) % iv == 0 for o in offsets]
            if any(ready):
                self._ready_point(done, None if all(ready) else ready, log)
        return self.best()
