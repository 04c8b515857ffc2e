"""Host-side checks that need no GPU: the C-ABI library loads and exports every
symbol the public header declares, the shard planner (pure host code) agrees
bit for bit with the oracle's independent planner, and argument errors are
reported as status codes before any launch."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import ws_oracle as O
from paper_2004_13336_b200 import binding as B
from paper_2004_13336_b200 import build as ws_build
from paper_2004_13336_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    ws_build.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "ws.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ws_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 18
    raw = C.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in ws.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_status_strings():
    L = B.lib()
    assert L.ws_status_string(0) == b"ok"
    for s in range(1, 8):
        assert len(L.ws_status_string(s)) > 0


@pytest.mark.parametrize("R", [1, 2, 3, 8, 10, 64, 1024])
@pytest.mark.parametrize("A", [8, 32, 128])
def test_planner_matches_oracle_planner(R, A):
    shapes = [(1,), (7,), (3, 3, 16, 32), (64, 128), (1031,), (5, 1, 9), (4096, 3)]
    plan = B.Plan(shapes, R, A, upload=False)
    ref = O.Plan([int(np.prod(s)) for s in shapes], R, A)
    assert (plan.S, plan.N, plan.T, plan.R, plan.A) == (ref.S, ref.N, ref.T, R, A)
    for t, sg in enumerate(plan.segments()):
        assert (sg.numel, sg.piece, sg.shard_off) == (ref.numel[t], ref.piece[t], ref.off[t])


def test_planner_on_model_shaped_workloads():
    for name in ("tiny", "resnet50", "transformer", "bert_large", "decoder_1p5b"):
        wl = W.WORKLOADS[name]()
        ref = O.Plan(wl.numels, wl.R, 32)
        for tile in (0, 2048, 8192):
            plan = B.Plan(wl.shapes, wl.R, 32, tile, upload=False)
            assert (plan.S, plan.N) == (ref.S, ref.N)
            segs = plan.segments()
            assert [s.piece for s in segs] == list(ref.piece)
            assert [s.shard_off for s in segs] == list(ref.off)
            if tile:    # tiles cover each piece exactly once, in order
                assert plan.ntiles == sum(-(-int(p) // tile) for p in ref.piece)
            else:       # default tile: between 1024 and 16384 elements
                lo = sum(-(-int(p) // 16384) for p in ref.piece)
                hi = sum(-(-int(p) // 1024) for p in ref.piece)
                assert lo <= plan.ntiles <= hi


def test_paper_worked_numbers_through_the_library():
    # Section 5.2 (4 MB / 2048 ways = 2 KB) and Section 4.1 ([3,3,256,256] at 8, 10 and 64 ways)
    p = B.Plan([(1024, 1024)], 2048, 8, upload=False)
    assert p.S * 4 == 2048
    assert B.Plan([(3, 3, 256, 256)], 64, 8, upload=False).S == 9216
    assert B.Plan([(3, 3, 256, 256)], 8, 8, upload=False).S == 73728
    assert B.Plan([(3, 3, 256, 256)], 10, 32, upload=False).S * 10 <= 10 * 256 * 256


def test_plan_create_rejects_bad_arguments():
    L = B.lib()
    d = (B.ws_tensor_desc * 1)()
    d[0].ndim = 1
    d[0].dims[0] = 10
    h = C.c_void_p()
    assert L.ws_plan_create(d, 1, 0, 32, 0, C.byref(h)) == 1          # R < 1
    assert L.ws_plan_create(d, 1, 4, 12, 0, C.byref(h)) == 1          # A not a power of two
    assert L.ws_plan_create(d, 1, 4, 4, 0, C.byref(h)) == 1           # A < 8
    assert L.ws_plan_create(d, 0, 4, 32, 0, C.byref(h)) == 1          # empty list
    assert L.ws_plan_create(d, 1, 4, 32, 1000, C.byref(h)) == 1       # tile not a multiple of 1024
    assert L.ws_plan_create(None, 1, 4, 32, 0, C.byref(h)) == 1
    d[0].dims[0] = -3
    assert L.ws_plan_create(d, 1, 4, 32, 0, C.byref(h)) == 1          # negative dimension
    assert not h.value


def test_empty_tensors_take_no_room():
    # a zero dimension makes an empty tensor: no piece, no tiles, neighbours unaffected
    shapes = [(5, 7), (0,), (3, 0, 4), (100,)]
    plan = B.Plan(shapes, 4, 8, upload=False)
    ref = O.Plan([35, 0, 0, 100], 4, 8)
    assert (plan.S, plan.N) == (ref.S, ref.N) == (16 + 32, 135)
    segs = plan.segments()
    assert [s.piece for s in segs] == [16, 0, 0, 32] == list(ref.piece)
    assert [s.shard_off for s in segs] == [0, 16, 16, 16] == list(ref.off)
    assert plan.arena_offsets() == [0, 40, 40, 40] and plan.arena_elems == 144


def test_calls_fail_cleanly_before_upload():
    # no device buffer yet: every data call must refuse without touching CUDA
    L = B.lib()
    plan = B.Plan([(64,)], 2, 8, upload=False)
    ptrs = (C.c_void_p * 1)(16)
    assert L.ws_pack(plan.handle, ptrs, 0, 16, None) == 5
    assert L.ws_unpack(plan.handle, 16, 0, ptrs, None) == 5
    g = B.ws_grads(C.cast((C.c_void_p * 2)(16, 16), C.POINTER(C.c_void_p)), 2, 0, 0)
    s = B.ws_state(16, 16, 16)
    hy = B.make_hyper("adam", W.tiny().hyper)
    assert L.ws_shard_update(plan.handle, 0, C.byref(g), C.byref(s), C.byref(hy), None, None, 0, None) == 5
    assert L.ws_shard_update(None, 0, C.byref(g), C.byref(s), C.byref(hy), None, None, 0, None) == 1
    assert plan.workspace_bytes("adam") == 0 and plan.workspace_bytes("sgdm") == 0
    assert plan.workspace_bytes("lamb") >= 4 * 1 + 16 * 1 + 8 * 2 * plan.ntiles


def test_planner_fuzz_against_oracle():
    # random tensor lists, shard counts, alignments, tile sizes and both layouts: the host planner and
    # the oracle's planners must agree on every offset, and the tiles must cover every shard exactly
    rng = np.random.default_rng(2004)
    for case in range(120):
        T = int(rng.integers(1, 40))
        numel = [int(x) for x in rng.choice([0, 1, 2, 7, 8, 31, 32, 33, 255, 1000, 4097, 70001], T)]
        R = int(rng.choice([1, 2, 3, 5, 8, 16, 33, 128, 1024]))
        A = int(rng.choice([8, 16, 32, 64, 256]))
        tile = int(rng.choice([0, 1024, 2048, 4096]))
        shapes = [(n,) for n in numel]
        per = B.Plan(shapes, R, A, tile, upload=False)
        ref = O.Plan(numel, R, A)
        assert (per.S, per.N) == (ref.S, ref.N)
        assert [(s.piece, s.shard_off) for s in per.segments()] == list(zip(ref.piece.tolist(), ref.off.tolist()))
        cat = B.Plan(shapes, R, A, tile, upload=False, layout="concat")
        fref = O.FlatPlan(numel, R, A)
        assert (cat.S, cat.N) == (fref.S, fref.N)
        assert [s.shard_off for s in cat.segments()] == fref.cat[:-1].tolist()
        assert cat.G <= per.G
        k = tile or 8192
        assert cat.ntiles >= R * (-(-cat.S // k)) if cat.S else cat.ntiles == 0


def test_header_is_plain_c_and_links_from_c(tmp_path):
    """include/ws.h compiles as strict C99 and a C program linked against libws.so can plan
    (host-only entry points; the paper's worked sharding numbers are checked inside it)."""
    import subprocess
    exe = tmp_path / "abi_host_check"
    src = os.path.join(ROOT, "tests", "c", "abi_host_check.c")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           src, "-o", str(exe), "-L", os.path.dirname(B.LIB_PATH), "-lws", f"-Wl,-rpath,{os.path.dirname(B.LIB_PATH)}"]
    subprocess.run(cmd, check=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "piece 73728" in r.stdout and "piece 9216" in r.stdout


def test_factored_layout_matches_oracle_view():
    # Adafactor's matrix view of every tensor (rows = leading dimensions together, cols = last one)
    shapes = [(5, 7), (0,), (3, 0, 4), (100,), (2, 3, 4, 5), (1,), (9, 1), (1, 9)]
    plan = B.Plan(shapes, 4, 8, upload=False)
    rows, cols, foff, tot = O.factor_shapes(shapes)
    assert plan.factored_elems == tot == 12 + 0 + 0 + 100 + 29 + 1 + 10 + 10
    assert plan.factored_layout() == list(zip(foff.tolist(), rows.tolist(), cols.tolist()))
    assert plan.workspace_bytes("adafactor") >= plan.workspace_bytes("lars") + 8 * tot + 4 * plan.T


@pytest.mark.parametrize("layout", ["per_tensor", "concat"])
@pytest.mark.parametrize("R,tile", [(1, 0), (3, 1024), (16, 4096), (40, 0)])
def test_one_launch_schedule_invariants(layout, R, tile):
    """The execution order of the one-kernel LAMB / LARS update (host logic): every element of every shard
    is covered by exactly one item, every item appears once per phase, an item's phase 2 comes after ALL
    phase-1 items of its tensor (the ratio needs every shard's partial sums, Section 4.1) and, except in
    the tail of the order, at least 512 entries after the last of them (no CTA waits for a ratio)."""
    shapes = [(1,), (7,), (3, 3, 16, 32), (64, 128), (0,), (1031,), (4099, 3), (300, 301), (32,), (70001,),
              (512, 1024), (1024, 2048), (1024,), (9,)]
    plan = B.Plan(shapes, R, 32, tile, upload=False, layout=layout)
    order, items = plan.schedule()
    n = len(items)
    assert len(order) == 2 * n and B.lib().ws_plan_schedule_bytes(plan.handle) >= 32 * n + 8 * n + 8 * len(shapes)
    # coverage of the [R][S] layout
    cover = np.zeros(plan.G, dtype=np.int32)
    numels = [int(np.prod(s)) for s in shapes]
    valid = 0
    for it in items:
        assert 0 < it.len <= 8192 and it.len % 8 == 0 and it.pos % 8 == 0 and 0 <= it.nvalid <= it.len
        assert it.nvalid == min(max(numels[it.tensor] - it.tensor_off, 0), it.len)
        cover[it.shard * plan.S + it.pos: it.shard * plan.S + it.pos + it.len] += 1
        valid += it.nvalid
    assert (cover == 1).all() and valid == plan.N
    # items are numbered tensor by tensor
    tens = [it.tensor for it in items]
    assert tens == sorted(tens)
    # each item once per phase; phase 2 after every phase-1 item of the tensor
    pos1, pos2 = {}, {}
    for p, (i, ph) in enumerate(order):
        d = pos1 if ph == 0 else pos2
        assert i not in d
        d[i] = p
    assert len(pos1) == len(pos2) == n
    last1 = {}
    for i, p in pos1.items():
        last1[tens[i]] = max(last1.get(tens[i], -1), p)
    early = 0
    for i, p in pos2.items():
        assert p > last1[tens[i]]
        if p - last1[tens[i]] < 512:
            early += 1
    # phase-1 items run in item order (tickets are handed out in this order); phase 2 takes the groups of
    # tensors in the same order but walks each group back to front (its last items are the freshest in L2):
    # the sequence is a chain of descending runs, each a contiguous block of indices, blocks ascending
    assert [i for i, ph in order if ph == 0] == list(range(n))
    seq2 = [i for i, ph in order if ph == 1]
    assert sorted(seq2) == list(range(n))
    lo_expected, k = 0, 0
    while k < n:
        hi = seq2[k]
        j = k
        while j + 1 < n and seq2[j + 1] == seq2[j] - 1:
            j += 1
        assert seq2[j] == lo_expected and hi >= seq2[j]
        lo_expected = hi + 1
        k = j + 1
    assert lo_expected == n
    # only the tail (after the last phase-1 entry) may hold phase-2 items that follow their tensor closely
    end1 = max(pos1.values())
    assert all(p > end1 for i, p in pos2.items() if p - last1[tens[i]] < 512)


def test_one_launch_schedule_on_bert_large_keeps_phase_two_close():
    """On the BERT-large set (R = 16) the state a phase-2 item reads was written a bounded distance earlier:
    except for the embedding (larger than L2) and the few tensors whose phase 2 queues behind the
    embedding's, the phase-1 to phase-2 distance of an item, in bytes of state touched in between (by either
    phase, so each byte counts twice), stays below 260 MB - the few hundred work items that are in flight
    at any time, 8192 elements each."""
    wl = W.bert_large()
    plan = B.Plan(wl.shapes, wl.R, 32, upload=False)
    order, items = plan.schedule()
    n = len(items)
    touched = np.cumsum([12 * items[i].len for i, _ in order])       # bytes of state moved up to entry p
    p1 = np.zeros(n, dtype=np.int64)
    p2 = np.zeros(n, dtype=np.int64)
    for p, (i, ph) in enumerate(order):
        (p1 if ph == 0 else p2)[i] = p
    dist = touched[p2] - touched[p1]
    big = np.array([wl.numels[it.tensor] * 12 > 200e6 for it in items])
    # (phase 2 walks a group back to front: the items written last are read first - a tenth of all items at
    # less than 100 MB - and the first-written ones last)
    assert np.quantile(dist[~big], 0.98) < 260e6
    assert np.median(dist[~big]) < 160e6
    assert np.quantile(dist[~big], 0.10) < 100e6
    assert plan.workspace_bytes("lamb") <= 4 * 1024 * 1024            # fits the library's static scratch


def test_build_tracks_every_header_the_kernels_include():
    """A change to any header of the kernel sources (.h and .cuh, and the public ws.h) must recompile every
    object: objects built against different versions of a shared struct would still link."""
    import re
    from paper_2004_13336_b200 import build as WB
    tracked = {os.path.basename(h) for h in WB._headers()}
    csrc = os.path.join(ROOT, "paper_2004_13336_b200", "csrc")
    included = set()
    for f in os.listdir(csrc):
        if f.endswith((".cu", ".cuh", ".h")):
            with open(os.path.join(csrc, f)) as fh:
                included |= set(re.findall(r'#include\s+"([^"]+)"', fh.read()))
    assert included and {os.path.basename(i) for i in included} <= tracked
