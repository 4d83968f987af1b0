"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, sizes its workspace sensibly and rejects bad arguments
before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import build as sk_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    sk_build.build()
    return sk.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "snapkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(snapkv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(L, name), name
    assert set(names) == set(sk.SYMBOLS)


def test_status_strings(L):
    assert sk.status_string(0) == "SNAPKV_OK"
    assert sk.status_string(5) == "SNAPKV_ERR_TIMEOUT"
    assert sk.status_string(77) == "SNAPKV_UNKNOWN_STATUS"


def test_out_rows(L):
    assert sk.snapkv_out_rows(1000, 256) == 256
    assert sk.snapkv_out_rows(1000, 1000) == 1000
    assert sk.snapkv_out_rows(1000, 5000) == 1000


def test_workspace_size(L):
    # votes alone are B*Hq*n fp32; the rest (statistics partials, counters) is small
    B, Hq, Hkv, Lp, d, W = 4, 32, 8, 32768, 128, 32
    ws = sk.snapkv_workspace_size(B, Hq, Hkv, Lp, d, W, 5, 1, 4096)
    votes = B * Hq * (Lp - W) * 4
    assert votes < ws < votes + (8 << 20)
    # rows longer than the on-chip key buffer need a second row-sized scratch
    ws4 = sk.snapkv_workspace_size(1, 32, 32, 380000, 128, 32, 7, 0, 4096)
    assert ws4 > 2 * 32 * (380000 - 32) * 4
    for bad in [(0, 4, 4, 100, 64, 8, 7, 0, 32), (1, 4, 3, 100, 64, 8, 7, 0, 32),
                (1, 4, 4, 100, 96, 8, 7, 0, 32), (1, 4, 4, 100, 64, 8, 4, 0, 32),
                (1, 4, 4, 100, 64, 8, 7, 2, 32), (1, 4, 4, 100, 64, 8, 7, 0, 8),
                (1, 4, 4, 100, 64, 200, 7, 0, 300), (1, 4, 4, 100, 64, 101, 7, 0, 300)]:
        assert sk.snapkv_workspace_size(*bad) == 0, bad
    assert sk.lib().snapkv_pool_topk_workspace_size(4, 1000) == 0
    # long rows: one key per vote plus small per-row histograms and counters
    assert 4 * 100000 * 4 < sk.lib().snapkv_pool_topk_workspace_size(4, 100000) < 4 * 100000 * 4 + (1 << 16)
    assert sk.snapkv_host_staging_size(1, 4, 4, 1024, 64, 32, 7, 0, 256) > 2 * 4 * 1024 * 64 * 2


FAKE = 0x1000  # non-null, 16-byte aligned, never dereferenced: validation fails first


def _compress(L, q=FAKE, k=FAKE, v=FAKE, B=1, Hq=4, Hkv=4, Lp=1024, d=64, W=32, pk=7, pt=0, budget=256,
              ok=FAKE, ov=FAKE, oi=FAKE, ws=None, wsb=0):
    return L.snapkv_compress(q, k, v, B, Hq, Hkv, Lp, d, W, pk, pt, budget, ok, ov, oi, ws, wsb, None)


def test_compress_rejects_bad_arguments_on_the_host(L):
    INV, UNS, WSP = 1, 2, 3
    assert _compress(L, B=0) == INV
    assert _compress(L, Hq=6, Hkv=4) == INV
    assert _compress(L, W=2000) == INV            # window longer than the prompt
    assert _compress(L, budget=32) == INV         # budget must exceed the window
    assert _compress(L, pk=6) == INV              # even pooling kernel
    assert _compress(L, pk=0) == INV
    assert _compress(L, pt=3) == INV
    assert _compress(L, q=None) == INV
    assert _compress(L, ok=None) == INV
    assert _compress(L, k=FAKE + 2) == INV        # misaligned
    assert _compress(L, d=96) == UNS
    assert _compress(L, d=256) == UNS
    assert _compress(L, W=200, budget=300) == UNS
    assert _compress(L, pk=65) == UNS
    assert _compress(L) == WSP                    # no workspace
    assert _compress(L, ws=FAKE + 16, wsb=1 << 30) == WSP  # workspace not 256-byte aligned
    assert _compress(L, ws=0x10000, wsb=16) == WSP    # too small


def test_other_entry_points_reject_bad_arguments(L):
    assert L.snapkv_window_scores(FAKE, FAKE, 1, 4, 4, 32, 64, 32, FAKE, None, 0, None) == 1  # W == L
    assert L.snapkv_window_scores(FAKE, FAKE, 1, 4, 4, 64, 64, 32, None, None, 0, None) == 1
    assert L.snapkv_window_scores(FAKE, FAKE, 1, 4, 4, 64, 64, 32, FAKE, None, 0, None) == 3
    assert L.snapkv_pool_topk(FAKE, 2, 100, 7, 0, 0, FAKE, None, 0, None) == 1     # ksel < 1
    assert L.snapkv_pool_topk(FAKE, 2, 100, 7, 0, 101, FAKE, None, 0, None) == 1   # ksel > n
    assert L.snapkv_pool_topk(FAKE, 2, 100, 8, 0, 10, FAKE, None, 0, None) == 1
    assert L.snapkv_pool_topk(FAKE, 2, 100000, 7, 0, 10, FAKE, None, 0, None) == 3  # needs scratch
    assert L.snapkv_gather(FAKE, FAKE, FAKE, 1, 4, 4, 100, 64, 8, 93, FAKE, FAKE, None) == 1  # ksel > n
    assert L.snapkv_gather(FAKE, FAKE, None, 1, 4, 4, 100, 64, 8, 10, FAKE, FAKE, None) == 1
    assert L.snapkv_compress_host(FAKE, FAKE, FAKE, 1, 4, 4, 1024, 64, 32, 7, 0, 256, FAKE, FAKE, FAKE,
                                  None, 0, None) == 3
    assert L.snapkv_compress_host(FAKE, FAKE, FAKE, 1, 4, 4, 1024, 96, 32, 7, 0, 256, FAKE, FAKE, FAKE,
                                  None, 0, None) == 2
    assert L.snapkv_device_status(None, None, None) == 1
    # supplied-normaliser variant: a missing or misaligned lse_obs is an argument error,
    # everything else is checked as in the functions it mirrors
    assert L.snapkv_window_scores_lse(FAKE, FAKE, None, 1, 4, 4, 1024, 64, 32, FAKE, FAKE, 1 << 30,
                                      None) == 1
    assert L.snapkv_window_scores_lse(FAKE, FAKE, FAKE + 2, 1, 4, 4, 1024, 64, 32, FAKE, FAKE,
                                      1 << 30, None) == 1
    assert L.snapkv_window_scores_lse(FAKE, FAKE, FAKE, 1, 4, 4, 1024, 64, 32, FAKE, None, 0,
                                      None) == 3
    assert L.snapkv_compress_lse(FAKE, FAKE, FAKE, None, 1, 4, 4, 1024, 64, 32, 7, 0, 256, FAKE, FAKE,
                                 FAKE, FAKE, 1 << 30, None) == 1
    assert L.snapkv_compress_lse(FAKE, FAKE, FAKE, FAKE, 1, 4, 4, 1024, 64, 32, 6, 0, 256, FAKE, FAKE,
                                 FAKE, FAKE, 1 << 30, None) == 1      # even pooling kernel
    assert L.snapkv_compress_lse(FAKE, FAKE, FAKE, FAKE, 1, 4, 4, 1024, 64, 32, 7, 0, 256, FAKE, FAKE,
                                 FAKE, None, 0, None) == 3


def test_strided_entry_point_checks_its_strides(L):
    import ctypes
    st = ctypes.c_int64 * 3
    dense = st(4 * 1024 * 64, 1024 * 64, 64)
    args = (None, 1, 4, 4, 1024, 64, 32, 7, 0, 256, FAKE, FAKE, FAKE)

    def call(ks, vs, ws=(FAKE, 1 << 30)):
        return L.snapkv_compress_strided(FAKE, FAKE, FAKE, ks, vs, *args, ws[0], ws[1], None)

    assert call(None, dense) == 1 and call(dense, None) == 1          # missing stride arrays
    assert call(st(4 * 1024 * 64, 1024 * 64, 60), dense) == 1         # not whole 16-byte vectors
    assert call(dense, st(4 * 1024 * 64, 1024 * 64, 56)) == 1         # rows would overlap
    assert call(st(0, 1024 * 64, 64), dense) == 1                     # zero stride
    assert call(dense, st(4 * 1024 * 64, -64, 64)) == 1               # negative stride
    assert call(st(1 << 39, 1024 * 64, 64), dense) == 1               # beyond a tensor map's reach
    # acceptable strides ([B, L, Hkv, d] order): the next check is the workspace
    assert call(st(1024 * 4 * 64, 64, 4 * 64), dense, (None, 0)) == 3


def test_varlen_entry_point_checks_every_sequence_before_launching(L):
    import ctypes
    i32, i64 = ctypes.c_int32 * 3, ctypes.c_int64 * 3
    tail = (None, 3, 4, 4, 1024, 64, 32, 7, 0, 256, FAKE, FAKE, FAKE)

    def call(lens, koff=None, ws=(FAKE, 1 << 30)):
        return L.snapkv_compress_varlen(FAKE, FAKE, FAKE, None, None, koff, None, lens, *tail,
                                        ws[0], ws[1], None)

    assert call(None) == 1                                  # no lengths
    assert call(i32(1024, 31, 500)) == 1                    # shorter than the window
    assert call(i32(1024, 1025, 500)) == 1                  # longer than Lmax
    assert call(i32(1024, 600, 500), i64(0, 4, 64)) == 1    # offset not a whole 16-byte vector
    assert call(i32(1024, 600, 500), i64(0, -8, 64)) == 1
    assert call(i32(1024, 600, 500), None, (None, 0)) == 3  # some sequence needs scratch
    assert call(i32(1024, 600, 500), None, (FAKE, 1024)) == 3


def test_hit_counts_rejects_bad_arguments(L):
    assert L.snapkv_hit_counts(None, FAKE, 4, 100, 10, 0.5, FAKE, None) == 1
    assert L.snapkv_hit_counts(FAKE, FAKE, 4, 100, 101, 0.5, FAKE, None) == 1   # k > n
    assert L.snapkv_hit_counts(FAKE, FAKE, 0, 100, 10, 0.5, FAKE, None) == 1
    assert L.snapkv_hit_counts(FAKE, FAKE, 70000, 100, 10, 0.5, FAKE, None) == 2


def test_decode_attention_rejects_bad_arguments(L):
    assert L.snapkv_decode_workspace_size(1, 4, 256, 96) == 0
    assert L.snapkv_decode_workspace_size(4, 32, 4096, 128) >= 4 * 32 * 130 * 4
    assert L.snapkv_decode_attention(FAKE, FAKE, FAKE, 1, 6, 4, 256, 128, FAKE, None, FAKE, 1 << 30, None) == 1
    assert L.snapkv_decode_attention(FAKE, FAKE, FAKE, 1, 4, 4, 256, 96, FAKE, None, FAKE, 1 << 30, None) == 2
    assert L.snapkv_decode_attention(FAKE, None, FAKE, 1, 4, 4, 256, 128, FAKE, None, FAKE, 1 << 30, None) == 1
    assert L.snapkv_decode_attention(FAKE, FAKE, FAKE, 1, 4, 4, 256, 128, FAKE, None, None, 0, None) == 3


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(sk, "_lib", None)
    monkeypatch.setattr(sk, "LIB_PATH", "/nonexistent/libsnapkv.so")
    with pytest.raises(sk.SnapKVError):
        sk.lib()


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2404_14469_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith(".py"):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+\S*oracle", text, flags=re.M), f
            elif f.endswith((".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read(), f
    assert "paper_2404_14469_b200" not in open(os.path.join(ROOT, "oracle", "snapkv_oracle.py")).read()
