"""Thin ctypes binding of libmetasd.so: argument marshalling only.

Every step of the draft-verify round runs inside the library's CUDA kernels; this module turns torch
tensors into raw device pointers and calls the C ABI declared in ``include/metasd.h`` under the same
names.  There is no CPU fallback: a missing library or a missing GPU raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmetasd.so")

BF16, FP32 = 0, 1
UCB, DUCB, SWUCB, EXP3, RAND, PETC = 0, 1, 2, 3, 4, 5
REWARD_BD, REWARD_BE = 0, 1
PATH_AUTO, PATH_STREAMING, PATH_FUSED = 0, 1, 2
ROWS_AUTO, ROWS_PLAIN, ROWS_STAGED, ROWS_BULK = 0, 1, 2, 3
STATUS_NONFINITE, STATUS_TOKEN_OOR, STATUS_Q_ZERO, STATUS_TIMEOUT, STATUS_BAD_POINTER, STATUS_BAD_LENGTH = 1, 2, 4, 8, 16, 32

OK, ERR_INVALID_ARGUMENT, ERR_UNSUPPORTED, ERR_CUDA, ERR_NO_MEMORY, ERR_BAD_STATE_BLOB = 0, -1, -2, -3, -4, -5

BANDITS = {"ucb": UCB, "ducb": DUCB, "swucb": SWUCB, "exp3": EXP3, "rand": RAND, "petc": PETC}
DTYPES = {"bf16": BF16, "fp32": FP32, torch.bfloat16: BF16, torch.float32: FP32}

EXPORTS = (
    "metasd_default_config", "metasd_init", "metasd_destroy", "metasd_reset", "metasd_select",
    "metasd_verify", "metasd_verify_host", "metasd_state_bytes", "metasd_state_export",
    "metasd_state_import", "metasd_last_status", "metasd_kernel_launches", "metasd_resolved_path",
    "metasd_strerror", "metasd_verify_noalloc", "metasd_set_draft_lengths", "metasd_state_validate",
    "metasd_resolved_row_kernel",
)


class MetasdConfig(C.Structure):
    """Mirror of ``metasd_config``."""
    _fields_ = [
        ("max_batch", C.c_int32), ("n_drafters", C.c_int32), ("max_draft", C.c_int32),
        ("vocab", C.c_int32), ("logit_dtype", C.c_int32), ("bandit", C.c_int32),
        ("reward", C.c_int32), ("window", C.c_int32), ("device", C.c_int32), ("path", C.c_int32),
        ("sequence_base", C.c_uint32), ("host_staging", C.c_int32),
        ("beta", C.c_double), ("gamma", C.c_double), ("reward_temperature", C.c_double),
        ("row_kernel", C.c_int32), ("row_threads", C.c_int32), ("row_stages", C.c_int32),
        ("keep_permille", C.c_int32), ("fused_cluster", C.c_int32), ("fused_threads", C.c_int32),
        ("wait_poll_limit", C.c_int32), ("row_cluster", C.c_int32),
    ]


class MetasdDiag(C.Structure):
    """Mirror of ``metasd_diag`` (20 bytes)."""
    _fields_ = [("p_x", C.c_float), ("q_x", C.c_float), ("D", C.c_float), ("u", C.c_float),
                ("accept", C.c_int32)]


class MetasdError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, strerror(code), code))
        self.code = code


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen libmetasd.so and declare the signatures.  Raises if the library has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            "%s is missing: build it with `python -m paper_2604_05417_b200.build` "
            "(there is no CPU fallback)" % path)
    lib = C.CDLL(path)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    lib.metasd_default_config.argtypes = [C.POINTER(MetasdConfig)]
    lib.metasd_default_config.restype = None
    lib.metasd_init.argtypes = [C.POINTER(vp), C.POINTER(MetasdConfig)]
    lib.metasd_destroy.argtypes = [vp]
    lib.metasd_destroy.restype = None
    lib.metasd_reset.argtypes = [vp, vp, i32, vp]
    lib.metasd_select.argtypes = [vp, i32, vp, vp]
    lib.metasd_verify.argtypes = [vp, i32, i32, vp, vp, vp, vp, i64, C.c_float, u64, vp, vp, vp, vp, vp]
    lib.metasd_verify_host.argtypes = [vp, i32, i32, vp, vp, vp, C.c_float, u64, vp, vp, vp, vp, vp]
    lib.metasd_state_bytes.argtypes = [vp]
    lib.metasd_state_bytes.restype = C.c_size_t
    lib.metasd_state_export.argtypes = [vp, vp, C.c_size_t, vp]
    lib.metasd_state_import.argtypes = [vp, vp, C.c_size_t, vp]
    lib.metasd_last_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    lib.metasd_kernel_launches.argtypes = [vp]
    lib.metasd_set_draft_lengths.argtypes = [vp, vp]
    lib.metasd_kernel_launches.restype = u64
    lib.metasd_resolved_path.argtypes = [vp, i32]
    lib.metasd_resolved_row_kernel.argtypes = [vp]
    lib.metasd_state_validate.argtypes = [C.POINTER(MetasdConfig), vp, C.c_size_t]
    lib.metasd_verify_noalloc.argtypes = [i32, i32, i32, i32, vp, vp, vp, C.c_float, C.c_float, i32, u64, C.c_uint32,
                                          C.c_uint32, vp, vp, vp, vp, vp]
    lib.metasd_strerror.argtypes = [C.c_int]
    lib.metasd_strerror.restype = C.c_char_p
    if path == LIB_PATH:
        _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().metasd_strerror(code).decode()


def default_config() -> MetasdConfig:
    cfg = MetasdConfig()
    load_library().metasd_default_config(C.byref(cfg))
    return cfg


def _check(code: int, what: str):
    if code != OK:
        raise MetasdError(code, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(device) -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream(device).cuda_stream)


@dataclass
class VerifyResult:
    accepted_len: torch.Tensor   # [B] int32
    next_token: torch.Tensor     # [B] int32
    reward: torch.Tensor         # [B] fp32
    diag: Optional[torch.Tensor] = None   # [B, k, 5] fp32 view: p_x, q_x, D, u, accept (int32 bits)

    def diag_fields(self):
        """p_x, q_x, D, u as fp32 [B,k] and accept as int32 [B,k]."""
        d = self.diag
        return d[..., 0], d[..., 1], d[..., 2], d[..., 3], d[..., 4].contiguous().view(torch.int32)


class MetaSD:
    """One library context: B independent bandits + the verify round, on one CUDA device."""

    def __init__(self, max_batch: int, n_drafters: int, max_draft: int, vocab: int, dtype="bf16",
                 bandit="ucb", beta: float = 0.01, gamma: float = 0.975, window: int = 50,
                 reward: int = REWARD_BD, reward_temperature: float = 1.0, device: int = 0,
                 path: int = PATH_AUTO, sequence_base: int = 0, host_staging: bool = False, **tuning):
        """tuning: the configuration's tuning and test fields by name (row_kernel, row_threads, row_stages, row_cluster,
        keep_permille, fused_cluster, fused_threads, wait_poll_limit)."""
        self.lib = load_library()
        cfg = default_config()
        cfg.max_batch, cfg.n_drafters, cfg.max_draft, cfg.vocab = max_batch, n_drafters, max_draft, vocab
        cfg.logit_dtype = DTYPES[dtype]
        cfg.bandit = BANDITS[bandit] if isinstance(bandit, str) else int(bandit)
        cfg.beta, cfg.gamma, cfg.window = beta, gamma, window
        cfg.reward, cfg.reward_temperature = reward, reward_temperature
        cfg.device, cfg.path, cfg.sequence_base = device, path, sequence_base
        cfg.host_staging = 1 if host_staging else 0
        for name, value in tuning.items():
            if name not in ("row_kernel", "row_threads", "row_stages", "row_cluster", "keep_permille", "fused_cluster",
                            "fused_threads", "wait_poll_limit"):
                raise TypeError("unknown configuration field %r" % name)
            setattr(cfg, name, int(value))
        self.cfg = cfg
        self.device = torch.device("cuda", device)
        self._ctx = C.c_void_p()
        _check(self.lib.metasd_init(C.byref(self._ctx), C.byref(cfg)), "metasd_init")

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self.lib.metasd_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the three calls of a round ------------------------------------------------------------
    def reset(self, seq_ids: Optional[torch.Tensor] = None):
        n = 0 if seq_ids is None else seq_ids.numel()
        _check(self.lib.metasd_reset(self._ctx, _ptr(seq_ids), n, _stream(self.device)), "metasd_reset")

    def select(self, batch: Optional[int] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        batch = self.cfg.max_batch if batch is None else batch
        if out is None:
            out = torch.empty(batch, dtype=torch.int32, device=self.device)
        _check(self.lib.metasd_select(self._ctx, batch, _ptr(out), _stream(self.device)), "metasd_select")
        return out

    def verify(self, target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor],
               draft_tokens: torch.Tensor, temperature: float, seed: int,
               drafter_table: Optional[torch.Tensor] = None, token_arm_stride: int = 0,
               out: Optional[VerifyResult] = None, want_diag: bool = False) -> VerifyResult:
        """target_logits [B,k+1,V]; draft_logits [B,k,V] or None with drafter_table = int64 device
        tensor of K data pointers; draft_tokens [B,k] int32 (or [K,B,k] with token_arm_stride=B*k)."""
        B, kp1, V = target_logits.shape
        k = kp1 - 1
        if out is None:
            out = VerifyResult(torch.empty(B, dtype=torch.int32, device=self.device),
                               torch.empty(B, dtype=torch.int32, device=self.device),
                               torch.empty(B, dtype=torch.float32, device=self.device))
        if want_diag and out.diag is None:
            out.diag = torch.zeros((B, k, 5), dtype=torch.float32, device=self.device)
        rc = self.lib.metasd_verify(
            self._ctx, B, k, _ptr(target_logits), _ptr(draft_logits), _ptr(drafter_table),
            _ptr(draft_tokens), token_arm_stride, C.c_float(temperature), C.c_uint64(seed),
            _ptr(out.accepted_len), _ptr(out.next_token), _ptr(out.reward), _ptr(out.diag),
            _stream(self.device))
        _check(rc, "metasd_verify")
        return out

    def verify_host(self, target_logits: torch.Tensor, draft_logits: torch.Tensor,
                    draft_tokens: torch.Tensor, temperature: float, seed: int,
                    accepted_len: torch.Tensor, next_token: torch.Tensor, reward: torch.Tensor,
                    arm_next: Optional[torch.Tensor] = None):
        """All tensors live in HOST memory (pinned for asynchronous copies); blocks until done."""
        B, kp1, V = target_logits.shape
        rc = self.lib.metasd_verify_host(
            self._ctx, B, kp1 - 1, _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens),
            C.c_float(temperature), C.c_uint64(seed), _ptr(accepted_len), _ptr(next_token),
            _ptr(reward), _ptr(arm_next), _stream(self.device))
        _check(rc, "metasd_verify_host")

    # -- state ------------------------------------------------------------------------------------
    def state_export(self) -> bytes:
        n = self.lib.metasd_state_bytes(self._ctx)
        buf = C.create_string_buffer(n)
        _check(self.lib.metasd_state_export(self._ctx, buf, n, _stream(self.device)), "metasd_state_export")
        return buf.raw

    def state_import(self, blob: bytes):
        buf = C.create_string_buffer(blob, len(blob))
        _check(self.lib.metasd_state_import(self._ctx, buf, len(blob), _stream(self.device)), "metasd_state_import")

    def set_draft_lengths(self, draft_len: Optional[torch.Tensor]):
        """Registers an int32 device tensor [max_batch] of per-sequence draft lengths (None: all sequences draft k).
        The tensor is kept alive by this object and read by every later verify call."""
        if draft_len is not None:
            assert draft_len.dtype == torch.int32 and draft_len.is_cuda and draft_len.is_contiguous()
            assert draft_len.numel() >= self.cfg.max_batch
        self._draft_len = draft_len
        _check(self.lib.metasd_set_draft_lengths(self._ctx, None if draft_len is None else draft_len.data_ptr()),
               "metasd_set_draft_lengths")

    def last_status(self) -> int:
        flags = C.c_uint32()
        _check(self.lib.metasd_last_status(self._ctx, C.byref(flags), _stream(self.device)), "metasd_last_status")
        return flags.value

    def kernel_launches(self) -> int:
        return int(self.lib.metasd_kernel_launches(self._ctx))

    def resolved_path(self, k: int) -> int:
        return int(self.lib.metasd_resolved_path(self._ctx, k))

    def resolved_row_kernel(self) -> int:
        return int(self.lib.metasd_resolved_row_kernel(self._ctx))


def verify_noalloc(target_logits: torch.Tensor, draft_logits: torch.Tensor, draft_tokens: torch.Tensor,
                   temperature: float, seed: int, round_: int, accepted_len: torch.Tensor,
                   next_token: torch.Tensor, reward: torch.Tensor, status: Optional[torch.Tensor] = None,
                   sequence_base: int = 0, reward_temperature: float = 1.0, reward_kind: int = REWARD_BD) -> int:
    """metasd_verify_noalloc on the current device and stream: no context, no allocation inside the
    library; the caller provides every buffer.  Returns the library's error code."""
    B, kp1, V = target_logits.shape
    dev = target_logits.device
    return load_library().metasd_verify_noalloc(
        B, kp1 - 1, V, DTYPES[target_logits.dtype], _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens),
        C.c_float(temperature), C.c_float(reward_temperature), reward_kind, C.c_uint64(seed),
        C.c_uint32(sequence_base), C.c_uint32(round_), _ptr(accepted_len), _ptr(next_token), _ptr(reward),
        _ptr(status), _stream(dev))


def state_validate(cfg: MetasdConfig, blob: bytes) -> int:
    """metasd_state_validate: the host-only check of a state blob (returns the library's error code)."""
    buf = C.create_string_buffer(blob, len(blob))
    return int(load_library().metasd_state_validate(C.byref(cfg), buf, len(blob)))


def pointer_table(tensors: Sequence[torch.Tensor]) -> torch.Tensor:
    """Device int64 tensor holding the data pointers of the K drafters' [B,k,V] logit tensors."""
    dev = tensors[0].device
    return torch.tensor([t.data_ptr() for t in tensors], dtype=torch.int64, device=dev)


def parse_state(blob: bytes, max_batch: int, n_drafters: int, window: int) -> dict:
    """Splits a state blob into numpy arrays (t, arm, stat_a, stat_b, win_arm, win_reward)."""
    import numpy as np
    B, K, tau = max_batch, n_drafters, window
    off = 24
    out = {"header": np.frombuffer(blob, dtype=np.int32, count=6).copy()}
    for name, dt, shape in (("t", np.int32, (B,)), ("arm", np.int32, (B,)), ("stat_a", np.float64, (B, K)),
                            ("stat_b", np.float64, (B, K)), ("win_arm", np.int32, (B, tau)),
                            ("win_reward", np.float64, (B, tau))):
        n = int(np.prod(shape))
        out[name] = np.frombuffer(blob, dtype=dt, count=n, offset=off).reshape(shape).copy()
        off += n * np.dtype(dt).itemsize
    return out


def pack_state(parts: dict) -> bytes:
    """Inverse of parse_state."""
    import numpy as np
    return b"".join([np.asarray(parts["header"], dtype=np.int32).tobytes()] +
                    [np.ascontiguousarray(parts[n]).tobytes()
                     for n in ("t", "arm", "stat_a", "stat_b", "win_arm", "win_reward")])
