"""The C-ABI library loads and exports every symbol include/*.h declares; host-side
argument checks and size queries work without a GPU (no compute call is made here)."""
import ctypes
import os
import re

import pytest

from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import build as sp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sp_build.build()
    return sp.load_library()


def test_header_symbols_are_exported(lib):
    inc = os.path.join(ROOT, "include")
    header = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(santapp_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(sp.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), f"{name} not exported"


def test_version_and_strerror(lib):
    assert lib.santapp_version() >= 100
    assert lib.santapp_strerror(0) == b"ok"
    assert b"invalid" in lib.santapp_strerror(sp.SANTAPP_ERR_INVALID_ARG)
    assert b"workspace" in lib.santapp_strerror(sp.SANTAPP_ERR_WORKSPACE_TOO_SMALL)


def test_sizes_follow_algorithms_4_and_2(lib):
    g = sp.Geometry(3, 28, 4, 128, 512, 32)
    s = sp.santapp_build_teams_sizes(g, [32768, 8192 + 100, 5])
    # ceil(N/P) parents; a parent of c rows gives min(R, c) teams
    assert s.rows_total == 32768 + 8292 + 5
    assert s.teams_total == 64 * 32 + (16 * 32 + 32) + 5
    assert s.max_teams_per_seq == 2048 and s.max_rows_per_seq == 32768
    assert s.team_row_start_elems == 4 * (s.teams_total + 3)
    assert s.build_workspace_bytes >= 2 * 4 * s.rows_total


@pytest.mark.parametrize("kw,status", [
    (dict(n_seqs=0), sp.SANTAPP_ERR_INVALID_ARG),
    (dict(n_q_heads=30), sp.SANTAPP_ERR_INVALID_ARG),            # Hkv must divide Hq
    (dict(reps_per_parent=7), sp.SANTAPP_ERR_INVALID_ARG),       # R must divide P
    (dict(head_dim=64), sp.SANTAPP_ERR_UNSUPPORTED),
    (dict(n_q_heads=36), sp.SANTAPP_ERR_UNSUPPORTED),            # 9 query heads per KV head
    (dict(parent_size=1024), sp.SANTAPP_ERR_UNSUPPORTED),
])
def test_bad_geometry_is_rejected_on_the_host(lib, kw, status):
    base = dict(n_seqs=1, n_q_heads=28, n_kv_heads=4, head_dim=128, parent_size=512, reps_per_parent=32)
    base.update(kw)
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_build_teams_sizes(sp.Geometry(**base), [1024] * max(base["n_seqs"], 1))
    assert e.value.status == status


def test_bad_prompt_length_is_rejected(lib):
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_build_teams_sizes(sp.Geometry(2, 28, 4), [1024, 0])
    assert e.value.status == sp.SANTAPP_ERR_INVALID_ARG


def test_null_arguments_return_invalid_arg_without_touching_a_gpu(lib):
    g = sp.Geometry(1, 28, 4).c()
    t = sp.CTeams()                                                # all null
    rc = lib.santapp_decode_attn(ctypes.byref(g), ctypes.byref(t), None, None, None, None, 0, 32, 0, 0, None, 0,
                                 0.0, None, None, None, 0, None)
    assert rc == sp.SANTAPP_ERR_INVALID_ARG
    rc = lib.santapp_dense_decode_attn(ctypes.byref(g), ctypes.byref(t), None, None, None, None, 0, 0.0, None,
                                       None, 0, None)
    assert rc == sp.SANTAPP_ERR_INVALID_ARG
    rc = lib.santapp_build_teams(ctypes.byref(g), (ctypes.c_int32 * 1)(1024), None, None, ctypes.byref(t), None, 0,
                                 None)
    assert rc == sp.SANTAPP_ERR_INVALID_ARG


def test_misaligned_pointers_are_refused_on_the_host(lib):
    """Device arrays are accessed 16 bytes at a time; a pointer that would fault there is refused
    before any launch (fake addresses: nothing is dereferenced)."""
    g = sp.Geometry(1, 28, 4).c()
    A = 0x10000                                                     # an aligned fake address
    t = sp.CTeams(A, A, A, A, A, A, A, A, A, 32768, 2048, 2048, 32768)
    args = dict(q=A, out=A, ws=A)

    def decode(q=A, out=A, ws=A, teams=t):
        return lib.santapp_decode_attn(ctypes.byref(g), ctypes.byref(teams), q, None, None, None, 0, 32, 0, 0, None,
                                       0, 0.0, out, None, ws, 0, None)

    assert decode(q=A + 2) == sp.SANTAPP_ERR_INVALID_ARG
    assert decode(out=A + 4) == sp.SANTAPP_ERR_INVALID_ARG
    assert decode(ws=A + 8) == sp.SANTAPP_ERR_INVALID_ARG
    bad = sp.CTeams(A + 2, A, A, A, A, A, A, A, A, 32768, 2048, 2048, 32768)
    assert decode(teams=bad) == sp.SANTAPP_ERR_INVALID_ARG
    # aligned pointers pass the checks and fail later only because the workspace is too small
    assert decode() == sp.SANTAPP_ERR_WORKSPACE_TOO_SMALL


def test_workspace_queries(lib):
    g = sp.Geometry(1, 28, 4)
    t = sp.CTeams(1, 1, 1, 1, 1, 1, 1, 1, 0, 32768, 8192, 2048, 32768)
    ws32 = lib.santapp_decode_workspace_bytes(ctypes.byref(g.c()), ctypes.byref(t), 32)
    ws64 = lib.santapp_decode_workspace_bytes(ctypes.byref(g.c()), ctypes.byref(t), 64)
    wsd = lib.santapp_dense_workspace_bytes(ctypes.byref(g.c()), ctypes.byref(t))
    assert 0 < wsd < ws32 < ws64 < 64 << 20
    assert ws32 >= 4 * 28 * 8192                                    # the fp32 perturbed scores
    assert lib.santapp_decode_workspace_bytes(ctypes.byref(g.c()), ctypes.byref(t), 0) == 0


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(sp.SantappError):
        sp.load_library(str(tmp_path / "libsantapp.so"))


@pytest.mark.parametrize("N,P,want", [(32768, 512, 64), (1000, 16, 62), (3, 16, 2), (5, 1, 5), (1, 16, 0), (8, 0, 0)])
def test_kmeans_parent_count_is_the_first_line_of_algorithm_3(lib, N, P, want):
    assert sp.santapp_kmeans_parent_count(N, P) == want


def test_parent_teams_sizes(lib):
    g = sp.Geometry(2, 28, 4, 128, 16, 4)
    sz = sp.santapp_parent_teams_sizes(g, [1000, 10], [62, 5])
    assert sz.rows_total == 1010
    assert sz.teams_total == 62 * 4 + 10              # min(N, parents * R) slots per sequence
    assert sz.max_teams_per_seq == 248 and sz.max_rows_per_seq == 1000
    assert sz.team_row_start_elems == 4 * (sz.teams_total + 2)
    assert sz.build_workspace_bytes > 25 * 4 * 1010
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_parent_teams_sizes(g, [1000, 10], [62, 0])
    assert e.value.status == sp.SANTAPP_ERR_INVALID_ARG


def test_parent_calls_refuse_null_and_misaligned_arguments(lib):
    g = sp.Geometry(1, 28, 4).c()
    n = (ctypes.c_int32 * 1)(1024)
    c = (ctypes.c_int32 * 1)(2)
    A = 0x10000
    t = sp.CTeams(A, A, A, A, A, A, A, A, A, 0, 0, 0, 0)
    assert lib.santapp_assign_parents(ctypes.byref(g), n, c, None, A, A, A, 1 << 20, None) == sp.SANTAPP_ERR_INVALID_ARG
    assert lib.santapp_assign_parents(ctypes.byref(g), n, c, A + 2, A, A, A, 1 << 20, None) == sp.SANTAPP_ERR_INVALID_ARG
    assert lib.santapp_assign_parents(ctypes.byref(g), n, c, A, A, A, A, 8, None) == sp.SANTAPP_ERR_WORKSPACE_TOO_SMALL
    assert lib.santapp_build_teams_parents(ctypes.byref(g), n, c, A, A, None, ctypes.byref(t), A, 1 << 30,
                                           None) == sp.SANTAPP_ERR_INVALID_ARG
    no_count = sp.CTeams(A, A, A, A, A, A, A, A, 0, 0, 0, 0, 0)
    assert lib.santapp_build_teams_parents(ctypes.byref(g), n, c, A, A, A, ctypes.byref(no_count), A, 1 << 30,
                                           None) == sp.SANTAPP_ERR_INVALID_ARG
    assert lib.santapp_build_teams_parents(ctypes.byref(g), n, c, A, A, A, ctypes.byref(t), A, 16,
                                           None) == sp.SANTAPP_ERR_WORKSPACE_TOO_SMALL


def test_kmeans_fit_argument_checks(lib):
    g = sp.Geometry(1, 28, 4).c()
    n = (ctypes.c_int32 * 1)(1024)
    k = (ctypes.c_int32 * 1)(8)
    A = 0x10000
    ok = sp.CKmeansOpts(256, 100, 10, 0, 0.01, 0, 0, 0)
    need = lib.santapp_kmeans_fit_workspace_bytes(ctypes.byref(g), n, k, ctypes.byref(ok))
    assert need > 4 * 1024 * 4                                     # at least the shuffle array
    for bad in (sp.CKmeansOpts(0, 100, 10, 0, 0.01, 0, 0, 0), sp.CKmeansOpts(256, 0, 10, 0, 0.01, 0, 0, 0),
                sp.CKmeansOpts(256, 100, 0, 0, 0.01, 0, 0, 0), sp.CKmeansOpts(256, 100, 10, 0, -1.0, 0, 0, 0)):
        assert lib.santapp_kmeans_fit_workspace_bytes(ctypes.byref(g), n, k, ctypes.byref(bad)) == 0
        assert lib.santapp_kmeans_fit(ctypes.byref(g), n, k, A, ctypes.byref(bad), A, None, A, 1 << 40,
                                      None) == sp.SANTAPP_ERR_INVALID_ARG
    big = sp.CKmeansOpts(8192, 100, 10, 0, 0.01, 0, 0, 0)
    assert lib.santapp_kmeans_fit(ctypes.byref(g), n, k, A, ctypes.byref(big), A, None, A, 1 << 40,
                                  None) == sp.SANTAPP_ERR_UNSUPPORTED
    too_many = (ctypes.c_int32 * 1)(2000)                           # more centres than keys
    assert lib.santapp_kmeans_fit(ctypes.byref(g), n, too_many, A, ctypes.byref(ok), A, None, A, 1 << 40,
                                  None) == sp.SANTAPP_ERR_INVALID_ARG
    assert lib.santapp_kmeans_fit(ctypes.byref(g), n, k, None, ctypes.byref(ok), A, None, A, 1 << 40,
                                  None) == sp.SANTAPP_ERR_INVALID_ARG
    assert lib.santapp_kmeans_fit(ctypes.byref(g), n, k, A + 2, ctypes.byref(ok), A, None, A, 1 << 40,
                                  None) == sp.SANTAPP_ERR_INVALID_ARG
    assert lib.santapp_kmeans_fit(ctypes.byref(g), n, k, A, ctypes.byref(ok), A, None, A, 64,
                                  None) == sp.SANTAPP_ERR_WORKSPACE_TOO_SMALL


def test_kmeans_fit_refuses_a_sample_that_does_not_fit_in_shared_memory(lib):
    g = sp.Geometry(1, 28, 4).c()
    n = (ctypes.c_int32 * 1)(200000)
    ok = sp.CKmeansOpts(4096, 100, 10, 0, 0.01, 0, 0, 0)
    fits = (ctypes.c_int32 * 1)(9514)
    too_many = (ctypes.c_int32 * 1)(9515)
    assert lib.santapp_kmeans_fit_workspace_bytes(ctypes.byref(g), n, fits, ctypes.byref(ok)) > 0
    assert lib.santapp_kmeans_fit(ctypes.byref(g), n, too_many, 0x10000, ctypes.byref(ok), 0x10000, None, 0x10000,
                                  1 << 40, None) == sp.SANTAPP_ERR_UNSUPPORTED


def test_latent_sizes_follow_algorithms_4_and_2(lib):
    g = sp.LatentGeometry(3, 16, 16, 4)
    s = sp.santapp_latent_sizes(g, [8192, 100, 5])
    assert s.rows_total == 8192 + 100 + 5
    assert s.teams_total == 512 * 4 + (6 * 4 + 4) + 4          # a tail of 4 rows gives 4 teams, of 5 rows min(R, 5)
    assert s.max_teams_per_seq == 2048 and s.max_rows_per_seq == 8192
    assert s.team_row_start_elems == s.teams_total + 3
    assert s.build_workspace_bytes >= s.rows_total


@pytest.mark.parametrize("geom,lens,status", [
    (sp.LatentGeometry(0, 16, 16, 4), [], sp.SANTAPP_ERR_INVALID_ARG),
    (sp.LatentGeometry(1, 0, 16, 4), [8], sp.SANTAPP_ERR_INVALID_ARG),
    (sp.LatentGeometry(1, 16, 16, 5), [8], sp.SANTAPP_ERR_INVALID_ARG),          # R must divide P
    (sp.LatentGeometry(1, 17, 16, 4), [8], sp.SANTAPP_ERR_UNSUPPORTED),          # more than 16 heads per row
    (sp.LatentGeometry(1, 16, 64, 4), [8], sp.SANTAPP_ERR_UNSUPPORTED),          # parents above 32 rows
    (sp.LatentGeometry(1, 16, 16, 4), [0], sp.SANTAPP_ERR_INVALID_ARG),
])
def test_bad_latent_geometry_is_rejected_on_the_host(lib, geom, lens, status):
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_latent_sizes(geom, lens)
    assert e.value.status == status
