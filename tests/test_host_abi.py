"""CPU-side checks of the boundary: the C-ABI library loads, exports every symbol the header declares, and the host
plan (tiling, quotas, workspace layout) agrees with the oracle's independent plan.  No compute call is made."""
import ctypes
import os
import re

import pytest

import oracle
import paper_2609_32628_b200 as da2
from paper_2609_32628_b200 import build as da2_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    da2_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "da2.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(da2_[a-z0-9_]+)\s*\(", header))
    assert {"da2_plan", "da2_prepare", "da2_attention_fwd", "da2_plan_info", "da2_device_status"} <= names
    lib = ctypes.CDLL(da2_build.LIB)
    for n in names:
        assert hasattr(lib, n), n


@pytest.mark.parametrize("cfg", [
    (1, 2, 4, 16, 16, 64, 0.0, 0.25, 0.25),
    (1, 12, 21, 30, 52, 128, 0.0, 0.10, 0.30),
    (1, 24, 33, 45, 80, 128, 0.0, 0.05, 0.20),
    (1, 40, 21, 45, 80, 128, 0.20, 0.40, 0.0),
])
@pytest.mark.parametrize("scope", [0, 1])
def test_plan_matches_oracle_plan(cfg, scope):
    B, H, T, Hg, Wg, d, f16, f8, f4 = cfg
    plan = da2.da2_plan(B, H, T, Hg, Wg, d, f16, f8, f4, rank_scope=scope)
    I = plan.info
    pl = oracle.plan(T, Hg, Wg)
    assert (I.R, I.S, I.N) == (pl.R, pl.S, pl.N)
    M = pl.R if scope == 0 else pl.R * pl.R
    k16, k8, k4 = oracle.quotas(f16, f8, f4, M)
    assert [int(x) for x in I.quota] == [k4, k8, k16]
    assert [int(x) for x in I.tier_active] == [int(k4 > 0), int(k8 > 0), int(k16 > 0)]
    assert I.ids_per_head >= (k4 + k8 + k16 if scope else (k4 + k8 + k16) * pl.R)
    # regions are disjoint, ordered and inside the workspace
    offs = [I.off_status, I.off_amax, I.off_vmax, I.off_gscale, *I.off_desc, *I.off_logits, I.off_map,
            I.off_counts, I.off_ids, I.off_select]
    assert offs == sorted(offs) and all(o % 256 == 0 for o in offs) and offs[-1] < I.workspace_bytes
    assert abs(I.softmax_scale - d ** -0.5) < 1e-7
    plan.close()


def test_plan_rejects_bad_arguments():
    ok = dict(B=1, H=1, T=1, Hg=8, Wg=8, head_dim=64, frac16=0.1, frac8=0.1, frac4=0.1)
    for bad, code in ((dict(head_dim=96), 2), (dict(frac8=0.95), 1), (dict(B=0), 1), (dict(lam=1.5), 1),
                      (dict(tile_h=16), 2), (dict(rank_scope=3), 1), (dict(T=400, Hg=64, Wg=64), 2),
                      (dict(g_q=[0.0]), 1)):
        with pytest.raises(da2.Da2Error) as e:
            da2.da2_plan(**{**ok, **bad})
        assert e.value.code == code, bad
    assert da2.da2_status_string(5) == "device-side wait timed out"


def test_compute_calls_reject_null_pointers_without_touching_cuda():
    plan = da2.da2_plan(1, 1, 1, 8, 8, 64, 0.0, 0.5, 0.0)
    lib = da2.load_library()
    assert lib.da2_prepare(plan.handle, None, None, None, None, 0, None) == 1
    assert lib.da2_attention_fwd(plan.handle, None, None, None, None, None, None) == 1
    assert lib.da2_prepare(plan.handle, 16, 16, 16, 256, 10, None) == 3   # workspace too small, still no launch
    assert lib.da2_refresh_operands(plan.handle, None, None, None, None, 0, None) == 1
    assert lib.da2_refresh_operands(plan.handle, 16, 16, 16, 256, 10, None) == 3


@pytest.mark.parametrize("grid", [(2, 30, 52), (1, 45, 80), (3, 12, 20), (1, 9, 13), (2, 16, 16)])
@pytest.mark.parametrize("mode", ["tiles", "balanced", "tiles+prefix"])
def test_slot_table_matches_oracle(grid, mode):
    """The token-to-region map the kernels index with (fixed tiles, the balanced ragged partition of App. C.2, and
    prefix blocks) equals the oracle's independent table slot by slot; the balanced plan also reports the oracle's
    choice of band order and perimeter."""
    T, Hg, Wg = grid
    P = 77 if mode == "tiles+prefix" else 0
    plan = da2.da2_plan(1, 2, T, Hg, Wg, 64, 0.1, 0.2, 0.3, partition=1 if mode == "balanced" else 0, n_prefix=P)
    pl = oracle.plan_balanced(T, Hg, Wg, 64) if mode == "balanced" else oracle.plan(T, Hg, Wg)
    pl = oracle.plan_with_prefix(pl, P)
    I = plan.info
    assert I.R + I.R_prefix == pl.R and I.R == pl.R_video
    got = [[da2.da2_plan_slot_token(plan, a, j) for j in range(64)] for a in range(pl.R)]
    assert got == pl.slot_token.tolist()
    if mode == "balanced":
        assert (I.part_transposed, I.part_bands, I.part_perimeter) == oracle.plan_balanced(T, Hg, Wg, 64).choice
        assert I.R_f == -(-Hg * Wg // 64)
    assert da2.da2_plan_slot_token(plan, pl.R, 0) == -2 and da2.da2_plan_slot_token(plan, 0, 64) == -2
    plan.close()


def test_balanced_partition_rejects_other_capacities():
    with pytest.raises(da2.Da2Error) as e:
        da2.da2_plan(1, 1, 1, 16, 16, 64, 0.1, 0.1, 0.1, partition=1, capacity=128)
    assert e.value.code == 2
    with pytest.raises(da2.Da2Error) as e:
        da2.da2_plan(1, 1, 1, 16, 16, 64, 0.1, 0.1, 0.1, partition=2)
    assert e.value.code == 1
