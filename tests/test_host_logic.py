"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and
validates arguments on the host before any launch (no compute call is made here)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2606_24780_b200 import binding as b
from paper_2606_24780_b200 import build as bt_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    bt_build.build()
    return b.lib()


def test_exports_every_declared_symbol(lib):
    with open(os.path.join(ROOT, "include", "bt.h")) as f:
        text = f.read()
    declared = set(re.findall(r"\b(bt_[a-z0-9_]+)\s*\(", text))
    declared -= {"bt_model", "bt_status", "bt_config", "bt_adamw_config"}
    assert declared, "no declarations found"
    raw = ctypes.CDLL(b.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(raw, name), f"{name} declared in bt.h but not exported"
    assert declared == set(b.exported_symbols()), declared ^ set(b.exported_symbols())


def test_workspace_bytes_and_config_validation(lib):
    good = b.make_config(2, 64, 4, 64, 512, 512, 4)
    n = b.bt_workspace_bytes(good)
    assert n > 0 and n % 256 == 0
    bigger = b.make_config(2, 64, 4, 64, 512, 512, 8)
    assert b.bt_workspace_bytes(bigger) > n
    parts = b.bt_workspace_parts(good)
    assert sum(parts.values()) == n and all(v > 0 for v in parts.values())
    assert b.bt_workspace_parts(bigger)["params_grads_moments"] == parts["params_grads_moments"]
    assert b.bt_workspace_parts(bigger)["activations"] > parts["activations"]
    for bad in [b.make_config(0, 64, 4, 64, 512, 512, 4), b.make_config(2, 66, 4, 64, 512, 512, 4),
                b.make_config(2, 64, 4, 64, 512, 500, 4), b.make_config(2, 64, 4, 64, 512, 520, 4),
                b.make_config(2, 96, 4, 64, 512, 512, 4), b.make_config(2, 64, 4, 64, 512, 512, 0),
                b.make_config(2, 8192, 64, 64, 512, 512, 1)]:
        assert b.bt_workspace_bytes(bad) == 0
        assert lib.bt_last_error()


def test_null_and_misaligned_arguments_are_rejected(lib):
    cfg = b.make_config(2, 64, 4, 64, 512, 512, 4)
    with pytest.raises(b.BtError) as e:
        b.bt_model_create(cfg, None, 1 << 30, stream=0)
    assert e.value.status == 1
    with pytest.raises(b.BtError) as e:
        b.bt_model_create(cfg, 0x1001, 1 << 30, stream=0)
    assert e.value.status == 1
    with pytest.raises(b.BtError) as e:
        b.bt_model_create(cfg, 0x10000, 1024, stream=0)          # workspace too small
    assert e.value.status == 3
    with pytest.raises(b.BtError) as e:
        b.bt_op_gelu_fwd(0x1000, 6, 0, 0x2000, None, stream=0)   # n not a multiple of 4
    assert e.value.status == 1
    with pytest.raises(b.BtError) as e:
        b.bt_op_gelu_fwd(0x1004, 8, 0, 0x2000, None, stream=0)   # misaligned
    assert e.value.status == 1
    with pytest.raises(b.BtError) as e:
        b.bt_op_gemm(7, 128, 128, 128, 0x1000, 0x2000, 0x3000, None, None, 0x4000, 1 << 40, 0, stream=0)
    assert e.value.status == 1
    with pytest.raises(b.BtError) as e:
        b.bt_op_gemm(0, 128, 128, 128, 0x1000, 0x2000, 0x3000, None, None, 0x4000, 16, 0, stream=0)
    assert e.value.status == 3
    with pytest.raises(b.BtError) as e:
        b.bt_op_attention_fwd(0x1000, 1, 8, 48, 2, 0x2000, None, 0x3000, 0, stream=0)   # head_dim 24
    assert e.value.status == 2
    with pytest.raises(b.BtError) as e:
        b.bt_op_softmax_xent(0x1000, 0x2000, 4, 10, 0.25, 0x3000, None, None, None, stream=0)
    assert e.value.status == 1
    assert b.bt_op_gemm_scratch_bytes(0, 128, 128, 128) > 0
    assert b.bt_op_layernorm_bwd_scratch_bytes(1000, 768) > 0


def test_gemm_planner_choices(lib):
    """bt_op_gemm_plan is host arithmetic.  The projections with 768 output columns and a long K (96 pair
    tiles for 74 CTA pairs) get a tail split; the same width with K = 768 keeps 192-wide single-CTA tiles;
    products that fill their rounds are left alone; forcing single-CTA tiles rules the tail split out."""
    p = b.bt_op_gemm_plan(8192, 768, 3072, True)
    assert p["pair"] == 1 and p["bn"] == 256 and p["tail_tiles"] == 22 and p["tail_splits"] == 3 and p["tail_kbps"] * 3 >= 3072 // 16
    p = b.bt_op_gemm_plan(8192, 768, 768, True)
    assert p["pair"] == 0 and p["bn"] == 192 and p["tail_splits"] == 0
    p = b.bt_op_gemm_plan(8192, 2304, 768, True)
    assert p["pair"] == 1 and p["tail_splits"] == 0 and p["splits"] == 1
    p = b.bt_op_gemm_plan(8192, 768, 3072, True, b.BT_FLAG_GEMM_SINGLE)
    assert p["pair"] == 0 and p["tail_splits"] == 0
    p = b.bt_op_gemm_plan(768, 768, 8192, False)          # a weight gradient: few tiles, K split over all of them
    assert p["splits"] > 1 and p["tail_splits"] == 0
    # raster of the tiles: groups of 4 row tiles where a group's units fit among those in flight (few tile
    # columns), 16 with many tile columns (the LM head), never more than there are row tiles
    assert b.bt_op_gemm_plan(8192, 768, 3072, True)["group_m"] == 4
    assert b.bt_op_gemm_plan(8192, 2304, 768, True)["group_m"] == 4
    assert b.bt_op_gemm_plan(8192, 50304, 768, False)["group_m"] == 16
    assert b.bt_op_gemm_plan(50304, 768, 8192, False)["group_m"] == 4
    assert b.bt_op_gemm_plan(512, 50304, 768, False)["group_m"] == 2
    with pytest.raises(b.BtError):
        b.bt_op_gemm_plan(0, 768, 768)


def test_host_id_check(lib):
    """bt_first_invalid_id is what bt_train_step_host and the loader run on ids that are still on the
    host: the position of the first id outside [0, vocab), or -1."""
    import torch
    ids = torch.arange(0, 100, dtype=torch.int32)
    assert b.bt_first_invalid_id(ids, 100) == -1
    assert b.bt_first_invalid_id(ids, 99) == 99
    assert b.bt_first_invalid_id(ids, 1) == 1
    ids[17] = -1
    assert b.bt_first_invalid_id(ids, 1000) == 17
    ids[3] = 2 ** 31 - 1
    assert b.bt_first_invalid_id(ids, 2 ** 31 - 1) == 3
    assert b.bt_first_invalid_id(ids[:0], 5) == -1
    assert lib.bt_first_invalid_id(None, 4, 5) == -2 and lib.bt_first_invalid_id(ids.data_ptr(), 4, 0) == -2


def test_lr_schedule_matches_oracle():
    """bt_lr_at is host arithmetic: compared with the oracle's schedule on the paper's four numbers
    (max 6e-4, min 6e-5, warmup 715, 19,073 steps) and on degenerate schedules."""
    import oracle
    for mx, mn, wu, ms in [(6e-4, 6e-5, 715, 19073), (1e-3, 1e-4, 10, 100), (3e-4, 3e-4, 0, 50), (1e-3, 0.0, 5, 5)]:
        sched = b.bt_lr_schedule(mx, mn, wu, ms)
        for step in list(range(0, 25)) + [wu - 1, wu, wu + 1, (wu + ms) // 2, ms - 1, ms, ms + 1, 10 * ms + 3]:
            want = oracle.lr_schedule(step, np.float32(mx), np.float32(mn), wu, ms)
            assert abs(b.bt_lr_at(sched, step) - want) <= 1e-6 * mx, (mx, mn, wu, ms, step)


def test_loader_plan_matches_oracle_cursor():
    """bt_loader_plan is host arithmetic (the cursor of Algorithm 2): same windows as the oracle's."""
    import oracle
    B, T = 2, 8
    for world in (1, 2, 3):
        for lens in ([B * T * world * 4 + 1, B * T * world * 2 + 5, B * T * world + 1], [B * T * world + 1],
                     [1000, 517, 999]):
            if min(lens) < B * T * world + 1:
                continue
            for rank in range(world):
                assert b.bt_loader_plan(lens, B, T, rank, world, 50) == oracle.loader_windows(lens, B, T, rank, world, 50)
    with pytest.raises(b.BtError):
        b.bt_loader_plan([10], B, T, 0, 1, 1)            # shorter than one batch + 1
