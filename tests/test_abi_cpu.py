"""CPU checks of the C-ABI library: it builds, loads, exports every declared symbol, validates
arguments on the host, and fails loudly (no fallback) when there is no CUDA device."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2604_05417_b200 import binding as M
from paper_2604_05417_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return M.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "metasd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(metasd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(M.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_mirrors_match_the_header(lib):
    cfg = M.default_config()
    assert C.sizeof(M.MetasdConfig) == 12 * 4 + 3 * 8 + 8 * 4
    assert (cfg.row_kernel, cfg.row_threads, cfg.row_stages, cfg.keep_permille, cfg.wait_poll_limit) == (0, 0, 0, 0, 0)
    assert C.sizeof(M.MetasdDiag) == 20
    assert (cfg.bandit, cfg.reward, cfg.logit_dtype, cfg.path) == (M.UCB, M.REWARD_BD, M.BF16, M.PATH_AUTO)
    assert (cfg.beta, cfg.gamma, cfg.window, cfg.reward_temperature) == (0.01, 0.975, 50, 1.0)


def test_host_side_validation(lib):
    ctx = C.c_void_p()
    bad = []
    for field, value in [("max_batch", 0), ("max_batch", 70000), ("n_drafters", 0), ("n_drafters", 17),
                         ("max_draft", 0), ("max_draft", 17), ("vocab", 0), ("window", 0), ("device", -1),
                         ("beta", -1.0), ("gamma", 0.0), ("gamma", 1.5), ("reward_temperature", 0.0)]:
        cfg = M.default_config()
        setattr(cfg, field, value)
        bad.append((field, lib.metasd_init(C.byref(ctx), C.byref(cfg))))
        assert ctx.value is None
    assert all(code == M.ERR_INVALID_ARGUMENT for _, code in bad), bad
    for field, value in [("row_threads", -1), ("keep_permille", 1001), ("fused_cluster", 17), ("fused_threads", 33),
                         ("wait_poll_limit", -1), ("row_cluster", -1), ("row_cluster", 9)]:
        cfg = M.default_config()
        setattr(cfg, field, value)
        assert lib.metasd_init(C.byref(ctx), C.byref(cfg)) == M.ERR_INVALID_ARGUMENT, field
    for field, value in [("logit_dtype", 7), ("bandit", 6), ("reward", 2), ("path", 9), ("row_kernel", 4)]:
        cfg = M.default_config()
        setattr(cfg, field, value)
        assert lib.metasd_init(C.byref(ctx), C.byref(cfg)) == M.ERR_UNSUPPORTED
    assert lib.metasd_init(None, C.byref(M.default_config())) == M.ERR_INVALID_ARGUMENT
    assert lib.metasd_init(C.byref(ctx), None) == M.ERR_INVALID_ARGUMENT
    # NULL contexts are refused everywhere
    assert lib.metasd_select(None, 1, None, None) == M.ERR_INVALID_ARGUMENT
    assert lib.metasd_reset(None, None, 0, None) == M.ERR_INVALID_ARGUMENT
    assert lib.metasd_state_bytes(None) == 0
    assert lib.metasd_kernel_launches(None) == 0
    lib.metasd_destroy(None)
    assert M.strerror(M.ERR_CUDA).startswith("CUDA error")
    assert M.strerror(-99) == "unknown error"


def test_state_blobs_are_checked_on_the_host_before_anything_reaches_the_device(lib):
    """A blob whose header matches but whose payload holds an arm, a window entry or a round counter outside its
    range, or a statistic that is not finite, is refused: the kernels index and divide with those values."""
    import numpy as np
    B, K, tau = 3, 4, 5
    cfg = M.default_config()
    cfg.max_batch, cfg.n_drafters, cfg.window, cfg.bandit = B, K, tau, M.SWUCB
    good = dict(header=np.array([0x4D534453, 1, B, K, tau, M.SWUCB], dtype=np.int32),
                t=np.array([0, 7, 123], dtype=np.int32), arm=np.array([0, 3, 1], dtype=np.int32),
                stat_a=np.linspace(0, 1, B * K).reshape(B, K), stat_b=np.arange(B * K, dtype=np.float64).reshape(B, K),
                win_arm=np.tile(np.arange(tau, dtype=np.int32) % K, (B, 1)), win_reward=np.full((B, tau), 0.25))
    assert M.state_validate(cfg, M.pack_state(good)) == M.OK

    def corrupted(field, index, value):
        parts = {k: np.array(v, copy=True) for k, v in good.items()}
        parts[field][index] = value
        return M.state_validate(cfg, M.pack_state(parts))
    for field, index, value in [("t", 1, -1), ("t", 2, 0x7FFFFFFF), ("arm", 0, -1), ("arm", 1, K), ("arm", 2, 1 << 20),
                                ("win_arm", (0, 0), K), ("win_arm", (2, 4), -3), ("stat_a", (1, 1), float("nan")),
                                ("stat_a", (0, 3), float("inf")), ("stat_b", (2, 0), -1.0), ("stat_b", (0, 0), float("nan")),
                                ("win_reward", (1, 2), float("-inf"))]:
        assert corrupted(field, index, value) == M.ERR_BAD_STATE_BLOB, (field, index, value)
    for slot, value in [(0, 0), (1, 2), (2, B + 1), (3, K - 1), (4, tau + 1), (5, M.UCB)]:   # the header
        parts = {k: np.array(v, copy=True) for k, v in good.items()}
        parts["header"][slot] = value
        assert M.state_validate(cfg, M.pack_state(parts)) == M.ERR_BAD_STATE_BLOB
    blob = M.pack_state(good)
    assert M.state_validate(cfg, blob[:-1]) == M.ERR_INVALID_ARGUMENT      # too short
    assert lib.metasd_state_validate(C.byref(cfg), None, len(blob)) == M.ERR_INVALID_ARGUMENT
    assert lib.metasd_state_validate(None, blob, len(blob)) == M.ERR_INVALID_ARGUMENT


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_device_is_a_loud_failure_not_a_fallback(lib):
    with pytest.raises(M.MetasdError) as e:
        M.MetaSD(4, 2, 3, 1000)
    assert e.value.code == M.ERR_CUDA


def test_missing_library_is_a_loud_failure(tmp_path):
    with pytest.raises(FileNotFoundError):
        M.load_library(str(tmp_path / "libmetasd.so"))


def test_product_code_never_touches_the_oracle():
    """The package, the header and the benchmark's own arm must not import or link oracle/."""
    pkg = os.path.join(ROOT, "paper_2604_05417_b200")
    for base, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(base, f)).read()
                assert "oracle" not in text.lower() or f == "workloads.py", f
    text = open(os.path.join(pkg, "workloads.py")).read()
    assert "import oracle" not in text and "from oracle" not in text
