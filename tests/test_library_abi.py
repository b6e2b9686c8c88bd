"""CPU-side checks of the C-ABI library: it builds, loads, exports every declared symbol, and its host-side
argument validation answers without touching a GPU."""
import ctypes
import os
import re

import pytest

import paper_2602_11562_b200 as P
from paper_2602_11562_b200 import build as laser_build


@pytest.fixture(scope="module")
def lib():
    laser_build.build()
    return P.load_library()


def test_exports_every_declared_symbol(lib, repo_root):
    hdr = open(os.path.join(repo_root, "include", "laser.h")).read()
    names = re.findall(r"LASER_API\s+[\w\s\*]+?\b(laser_\w+)\s*\(", hdr)
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n


def test_config_struct_matches_header(repo_root):
    hdr = open(os.path.join(repo_root, "include", "laser.h")).read()
    body = re.search(r"typedef struct laser_config \{(.*?)\} laser_config;", hdr, re.S).group(1)
    fields = re.findall(r"^\s*(int32_t|float)\s+(\w+);", body, re.M)
    assert [f[1] for f in fields] == [f[0] for f in P.LaserConfig._fields_]
    assert ctypes.sizeof(P.LaserConfig) == 4 * len(fields)


def _cfg(**kw):
    base = dict(num_users=2, max_len=64, d_model=32, d_qk=16, num_heads=2, seg_size=16, num_gsta_layers=1,
                dtype="f32", total_cands=6, max_cands_per_user=3)
    base.update(kw)
    return P.make_config(**base)


def test_workspace_query_and_validation(lib):
    assert P.laser_workspace_bytes(_cfg()) > 0
    assert P.laser_host_workspace_bytes(_cfg()) > P.laser_workspace_bytes(_cfg())
    assert P.laser_workspace_bytes(_cfg(num_heads=3)) == 0          # H must divide d and d_qk
    assert P.laser_workspace_bytes(_cfg(seg_size=0)) == 0
    assert P.laser_workspace_bytes(_cfg(dtype=7)) == 0
    assert P.laser_workspace_bytes(_cfg(max_cands_per_user=9)) == 0  # larger than total
    assert P.laser_workspace_bytes(_cfg(path=P.PATH_TENSOR)) == 0    # tensor path is bf16-only
    # host-detectable errors come back as negative statuses before anything is launched
    cfg = _cfg()
    null = ctypes.c_void_p(0)
    rc = lib.laser_forward(ctypes.byref(cfg), null, null, null, null, null, null, null, null, null, null, null, 0, null)
    assert rc == -1
    assert P.laser_status_string(rc) == "invalid argument"
    assert "workspace" in P.laser_status_string(-3)


def test_workspace_regions_are_disjoint_and_followed_by_a_guard_gap(lib):
    for kw in (dict(), dict(dtype="bf16", path=P.PATH_SIMT),
               dict(num_users=3, max_len=512, d_model=64, d_qk=64, num_heads=4, seg_size=64, num_gsta_layers=2, dtype="bf16",
                    total_cands=600, max_cands_per_user=200, path=P.PATH_TENSOR),
               dict(num_users=40, max_len=256, d_model=64, d_qk=32, num_heads=2, seg_size=64, dtype="bf16", total_cands=40,
                    max_cands_per_user=1, path=P.PATH_STREAM)):
        cfg = _cfg(**kw)
        total = P.laser_workspace_bytes(cfg)
        regions = P.laser_workspace_regions(cfg)
        assert total > 0 and len(regions) >= 3 and regions[0][0] == 0
        end = 0
        for i, (off, size) in enumerate(regions):
            assert off % 256 == 0
            assert off >= end + (256 if i else 0)          # at least 256 untouched bytes after the previous region
            end = off + size
        assert end + 256 <= total
    assert P.laser_workspace_regions(_cfg())[0][1] == 256   # the status block comes first
    with pytest.raises(P.LaserError):
        P.laser_workspace_regions(_cfg(num_heads=3))


def test_host_transfer_size_query(lib):
    import torch
    # 4 users x 4096 rows of 128 bf16 features (256 bytes each): everything else is small next to the items.  Without
    # a pinned items pointer the route is the one for pageable memory: one copy per run of contiguous users.
    cfg = _cfg(num_users=4, max_len=4096, d_model=128, d_qk=32, seg_size=128, dtype="bf16", total_cands=8,
               max_cands_per_user=2)
    row = 256
    other = 4 * 4 + 5 * 4 + 8 * row + 2 * 128 * 32 * 2 + 128 * 128 * 2 + 3 * 128 * 128 * 2
    full = torch.full((4,), 4096, dtype=torch.int32)
    assert P.laser_host_transfer_bytes(cfg, full) == (4 * 4096 * row + other, 8 * row)      # one padded copy
    short = torch.tensor([4096, 100, 0, 4096], dtype=torch.int32)                           # two runs
    assert P.laser_host_transfer_bytes(cfg, short) == ((4096 + 100 + 4096) * row + other, 8 * row)
    # lengths outside [0, L] are clamped for the copy (the device reports them)
    bad = torch.tensor([-5, 100, 9999, 7], dtype=torch.int32)                               # two runs
    assert P.laser_host_transfer_bytes(cfg, bad) == ((100 + 4096 + 7) * row + other, 8 * row)
    # saving less than the fixed cost of the extra copies: the padded array travels in one piece
    nearly = torch.tensor([3000, 3000, 3000, 3000], dtype=torch.int32)
    assert P.laser_host_transfer_bytes(cfg, nearly)[0] == 4 * 4096 * row + other


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2602_11562_b200 import binding
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "library_path", lambda: str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()
