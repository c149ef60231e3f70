"""Randomised parity: shapes, paddings, base misalignments, dtypes, ragged lengths, value scales
and masked (-inf) entries drawn from a seeded generator; every call against the fp64 oracle."""
import numpy as np
import pytest
import torch

import helpers as H
from oracle import ref
from paper_2603_11243_b200 import binding as ssd

pytestmark = pytest.mark.gpu


def random_matrix(rng, rows, V, dtype):
    """A [rows, V] view into a wider, offset matrix: ld > V and an element-aligned base."""
    pad, col0 = int(rng.integers(0, 9)), int(rng.integers(0, 8))
    ld = V + pad + col0
    scale = float(rng.choice([0.3, 1.0, 4.0, 12.0]))
    x = rng.normal(size=(rows, ld)).astype(np.float32) * scale
    if rows and V > 2 and rng.random() < 0.5:            # some masked logits
        mask = rng.random(size=(rows, ld)) < 0.1
        mask[:, col0 + int(rng.integers(0, V))] = False  # never a whole row
        x[mask] = -np.inf
    t = torch.from_numpy(x).to(dtype)
    return t, col0, ld


def ragged(rng, B, hi):
    lens = rng.integers(0, hi + 1, size=B)
    if B > 1:
        lens[int(rng.integers(0, B))] = 0
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int64), lens


@pytest.mark.parametrize("seed", range(16))
def test_stage1_random(cuda_device, seed):
    rng = np.random.default_rng(1000 + seed)
    V = int(rng.choice([1, 2, 5, 17, 64, 129, 348, 777, 1025, 2051, 4097]))
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    off, lens = ragged(rng, int(rng.integers(1, 8)), 90)
    wide, col0, ld = random_matrix(rng, int(off[-1]), V, dtype)
    blank = int(rng.integers(0, V))
    cap = int(rng.integers(0, 40))
    tau = float(rng.uniform(0.05, 4.0))
    dev = cuda_device
    view = wide.to(dev)[:, col0:col0 + V]
    g, out = H.guarded_ctc_outputs(int(off[-1]), len(lens), dev)
    offd = torch.from_numpy(off).to(dev)
    ssd.ssd_ctc_draft(view, offd, blank, cap, V=V, out=out)
    gate = ssd.ssd_entropy_gate(out["frame_entropy"], offd, tau)
    torch.cuda.synchronize()
    g.check()
    H.check_gate_from_maxima(out, gate, tau)
    orc = H.oracle_stage1(H.storage_numpy(wide[:, col0:col0 + V].contiguous()), V, off, blank, cap, tau)
    H.compare_stage1(out, gate, orc, off, tau, require_all_margins=False)


@pytest.mark.parametrize("seed", range(16))
def test_stage2_random(cuda_device, seed):
    rng = np.random.default_rng(2000 + seed)
    V = int(rng.choice([1, 3, 40, 1000, 4099, 20001, 32000, 65537]))
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    B = int(rng.integers(1, 7))
    off, lens = ragged(rng, B, 30 if V > 10000 else 120)
    M = int(off[-1])
    wide, col0, ld = random_matrix(rng, M, V, dtype)
    ids = rng.integers(0, V, size=M).astype(np.int32)
    if M and rng.random() < 0.3:
        ids[int(rng.integers(0, M))] = V + 3                 # one out-of-range id
    for r in range(M):                                        # most draft tokens likely
        if 0 <= ids[r] < V and rng.random() < 0.8:
            wide[r, col0 + ids[r]] = 25.0
    tau = float(rng.choice([0.0, 0.05, 0.1, 0.2, 0.9]))
    skip = (rng.random(size=B) < 0.25).astype(np.uint8) if rng.random() < 0.5 else None
    dev = cuda_device
    view = wide.to(dev)[:, col0:col0 + V]
    code = ssd.BF16 if dtype == torch.bfloat16 else ssd.F32
    g, out = H.guarded_verify_outputs(M, B, dev, ssd.ssd_verify_workspace_bytes(B, M, V, code))
    skipd = None if skip is None else torch.from_numpy(skip).to(dev)
    offd, idsd = torch.from_numpy(off).to(dev), torch.from_numpy(ids).to(dev)
    ssd.ssd_verify(view, offd, idsd, tau, skip=skipd, V=V, out=out)
    torch.cuda.synchronize()
    g.check()
    orc = ref.verify(H.storage_numpy(wide[:, col0:col0 + V].contiguous()), V, off, ids,
                     float(np.float32(tau)), skip=skip)
    H.compare_stage2(out, orc, off, tau, skip=skip, require_all_margins=False)
    # the early-exit call decides the same (it falls back to the full kernel at these sizes
    # unless there are many rows)
    ee = ssd.ssd_verify_early_exit(view, offd, idsd, tau, skip=skipd, V=V)
    torch.cuda.synchronize()
    assert torch.equal(ee["accepted_len"], out["accepted_len"])
    assert torch.equal(ee["all_accepted"], out["all_accepted"])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("V", [50001, 55553, 56700, 100003, 152065])
def test_stage2_wide_odd_rows(cuda_device, V, dtype):
    """Rows around and above what one ring stage holds (one stage of ~100 KB per row, or two
    or three equal parts), odd lengths, padded and misaligned.  The grid is limited to 40 CTAs
    so that a couple of hundred rows already take the unsplit path."""
    rng = np.random.default_rng(V)
    B, o = 5, H.opts(ctas=40)
    off, lens = ragged(rng, B, 90)
    while off[-1] < 4 * 40 + 10:
        off, lens = ragged(rng, B, 90)
    M = int(off[-1])
    wide, col0, ld = random_matrix(rng, M, V, dtype)
    ids = rng.integers(0, V, size=M).astype(np.int32)
    for r in range(M):
        if rng.random() < 0.9:
            wide[r, col0 + ids[r]] = 25.0
    dev = cuda_device
    view = wide.to(dev)[:, col0:col0 + V]
    code = ssd.BF16 if dtype == torch.bfloat16 else ssd.F32
    g, out = H.guarded_verify_outputs(M, B, dev, ssd.ssd_verify_workspace_bytes(B, M, V, code, o))
    offd, idsd = torch.from_numpy(off).to(dev), torch.from_numpy(ids).to(dev)
    ssd.ssd_verify(view, offd, idsd, 0.1, V=V, out=out, opts=o)
    torch.cuda.synchronize()
    g.check()
    orc = ref.verify(H.storage_numpy(wide[:, col0:col0 + V].contiguous()), V, off, ids,
                     float(np.float32(0.1)))
    H.compare_stage2(out, orc, off, 0.1, require_all_margins=False)
    ee = ssd.ssd_verify_early_exit(view, offd, idsd, 0.1, V=V, opts=o)
    torch.cuda.synchronize()
    assert torch.equal(ee["accepted_len"], out["accepted_len"])
    assert bool((ee["rows_read"] >= 0).all().item())          # the position-major kernel ran
    gr = ssd.ssd_greedy_step(view, V=V, opts=o)
    torch.cuda.synchronize()
    want = ref.greedy_step(H.storage_numpy(wide[:, col0:col0 + V].contiguous()), V)
    np.testing.assert_array_equal(gr["next_token"].cpu().numpy(), want["next_token"])


@pytest.mark.parametrize("seed", range(12))
def test_greedy_random(cuda_device, seed):
    rng = np.random.default_rng(3000 + seed)
    V = int(rng.choice([1, 2, 33, 1000, 4099, 20001, 49152, 100003]))
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    R = int(rng.integers(1, 40 if V > 10000 else 300))
    wide, col0, ld = random_matrix(rng, R, V, dtype)
    dev = cuda_device
    out = ssd.ssd_greedy_step(wide.to(dev)[:, col0:col0 + V], V=V)
    torch.cuda.synchronize()
    orc = ref.greedy_step(H.storage_numpy(wide[:, col0:col0 + V].contiguous()), V)
    np.testing.assert_array_equal(out["next_token"].cpu().numpy(), orc["next_token"])
    assert np.abs(out["next_logp"].cpu().numpy().astype(np.float64) - orc["next_logp"]).max() <= H.FLOAT_TOL
    assert np.abs(out["row_lse"].cpu().numpy().astype(np.float64) - orc["row_lse"]).max() <= H.FLOAT_TOL


@pytest.mark.parametrize("seed", range(6))
def test_early_exit_random_large(cuda_device, seed):
    """Enough rows for the position-major kernel; random reject structure."""
    rng = np.random.default_rng(4000 + seed)
    V = int(rng.choice([257, 4099, 16384]))
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    B = int(rng.integers(5, 40))
    lens = rng.integers(20, 140, size=B)
    lens[int(rng.integers(0, B))] = 0
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    M = int(off[-1])
    while M < 8 * 148 + 100:                  # below that, rows are cut into column spans
        lens = lens + 40                      # and the call falls back to the full kernel
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        M = int(off[-1])
    wide, col0, ld = random_matrix(rng, M, V, dtype)
    ids = rng.integers(0, V, size=M).astype(np.int32)
    for r in range(M):
        if rng.random() < 0.97:
            wide[r, col0 + ids[r]] = 25.0
    tau = 0.1
    dev = cuda_device
    view = wide.to(dev)[:, col0:col0 + V]
    offd, idsd = torch.from_numpy(off).to(dev), torch.from_numpy(ids).to(dev)
    code = ssd.BF16 if dtype == torch.bfloat16 else ssd.F32
    out = ssd.alloc_early_exit_outputs(M, B, V, code, dev)
    out["token_logp"].fill_(float("nan"))
    ssd.ssd_verify_early_exit(view, offd, idsd, tau, V=V, out=out)
    torch.cuda.synchronize()
    orc = ref.verify(H.storage_numpy(wide[:, col0:col0 + V].contiguous()), V, off, ids, float(np.float32(tau)))
    lp = out["token_logp"].cpu().numpy().astype(np.float64)
    safe = np.abs(orc["token_logp"] - np.log(tau)) > H.MARGIN
    for b in range(B):
        s = slice(int(off[b]), int(off[b + 1]))
        if not safe[s].all():
            continue
        assert int(out["accepted_len"].cpu()[b]) == orc["accepted_len"][b]
        need = min(int(lens[b]), int(orc["accepted_len"][b]) + 1)
        seg = lp[s]
        assert not np.isnan(seg[:need]).any()
        read = ~np.isnan(seg)
        want = orc["token_logp"][s]
        fin = read & np.isfinite(want)
        assert np.abs(seg[fin] - want[fin]).max(initial=0.0) <= H.FLOAT_TOL
        np.testing.assert_array_equal(seg[read & ~np.isfinite(want)], want[read & ~np.isfinite(want)])
    assert (out["rows_read"].cpu().numpy() >= 0).all()


def _close_scaled(got, want, what):
    """fp32 outputs of magnitude 1e3..1e5 cannot be within 1e-4 of the fp64 value: allow two
    fp32 ulps of the value on top of the absolute tolerance."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    fin = np.isfinite(want)
    tol = H.FLOAT_TOL + 2.5e-7 * np.abs(want[fin])
    assert (np.abs(got[fin] - want[fin]) <= tol).all(), what
    np.testing.assert_array_equal(got[~fin], want[~fin])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [60.0, 400.0, 3.0e4])
def test_huge_dynamic_range_takes_the_redo_paths(cuda_device, dtype, scale):
    """Logits hundreds to tens of thousands of nats apart: sums relative to a lane's first
    element overflow, so the kernels must fall back to their exact two-pass redo."""
    rng = np.random.default_rng(int(scale))
    dev = cuda_device
    V1, V2 = 1025, 20001
    x1 = torch.from_numpy((rng.normal(size=(70, V1)) * scale).astype(np.float32)).to(dtype)
    x1[:, :8] = -scale * 4                      # lanes whose first chunk is far below the maximum
    off = torch.tensor([0, 30, 70], dtype=torch.int64)
    out = ssd.ssd_ctc_draft(x1.to(dev), off.to(dev), 0, 50)
    torch.cuda.synchronize()
    o1 = ref.ctc_draft(H.storage_numpy(x1), V1, off.numpy(), 0, 50)
    np.testing.assert_array_equal(out["frame_argmax"].cpu().numpy(), o1["frame_argmax"])
    np.testing.assert_array_equal(out["draft_len"].cpu().numpy(), o1["draft_len"])
    _close_scaled(out["frame_lse"].cpu().numpy(), o1["frame_lse"], "frame_lse")
    _close_scaled(out["frame_entropy"].cpu().numpy(), o1["frame_entropy"], "frame_entropy")
    x2 = torch.from_numpy((rng.normal(size=(40, V2)) * scale).astype(np.float32)).to(dtype)
    x2[:, :4096] = -scale * 4
    ids = torch.from_numpy(rng.integers(0, V2, size=40).astype(np.int32))
    ids[::3] = torch.from_numpy(np.argmax(x2.float().numpy()[::3], axis=1).astype(np.int32))
    off2 = torch.tensor([0, 15, 40], dtype=torch.int64)
    v = ssd.ssd_verify(x2.to(dev), off2.to(dev), ids.to(dev), 0.1)
    gr = ssd.ssd_greedy_step(x2.to(dev))
    torch.cuda.synchronize()
    o2 = ref.verify(H.storage_numpy(x2), V2, off2.numpy(), ids.numpy(), float(np.float32(0.1)))
    _close_scaled(v["row_lse"].cpu().numpy(), o2["row_lse"], "row_lse")
    _close_scaled(v["token_logp"].cpu().numpy(), o2["token_logp"], "token_logp")
    np.testing.assert_array_equal(v["accepted_len"].cpu().numpy(), o2["accepted_len"])
    og = ref.greedy_step(H.storage_numpy(x2), V2)
    np.testing.assert_array_equal(gr["next_token"].cpu().numpy(), og["next_token"])
    _close_scaled(gr["next_logp"].cpu().numpy(), og["next_logp"], "next_logp")
    _close_scaled(gr["row_lse"].cpu().numpy(), og["row_lse"], "greedy row_lse")


@pytest.mark.parametrize("seed", range(40))
def test_early_exit_against_verify_random_options(cuda_device, seed):
    """Random shapes, thresholds, skip flags and launch options (grid, warps, ring): the same
    decisions as ssd_verify, its log-likelihoods up to each first reject, and no status bit that
    ssd_verify does not report (bits of rows after a first reject may be missing: not read)."""
    rng = np.random.default_rng(7000 + seed)
    V = int(rng.choice([33, 257, 1000, 4099, 8192, 16384]))
    dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
    B = int(rng.choice([1, 2, 7, 32, 33, 257, 2049]))
    lens = rng.integers(0, int(rng.choice([3, 10, 60, 200])) + 1, size=B)
    ctas = int(rng.choice([0, 8, 37]))
    while lens.sum() < 4 * (ctas if ctas else 148) + 5:
        lens = lens + 1 + rng.integers(0, 3, size=B)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    M = int(off[-1])
    dev = cuda_device
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    pad = int(rng.integers(0, 9))
    col0 = int(rng.integers(0, pad + 1))
    wide = (torch.randn((M, V + pad), generator=g, device=dev) * 2).to(dtype)
    ids = torch.randint(0, V, (M,), generator=g, device=dev, dtype=torch.int32)
    keep = torch.rand((M,), generator=g, device=dev) < float(rng.choice([0.9, 0.97, 0.995, 1.0]))
    rows = torch.arange(M, device=dev)[keep]
    wide[rows, col0 + ids[rows].long()] = 30.0
    if rng.random() < 0.3:
        ids[int(rng.integers(0, M))] = V + 3
    view = wide[:, col0:col0 + V]
    offd = torch.from_numpy(off).to(dev)
    skip = (torch.rand((B,), generator=g, device=dev) < 0.3).to(torch.uint8) if rng.random() < 0.5 else None
    kw = {}
    if ctas:
        kw["ctas"] = ctas
    if rng.random() < 0.4:
        kw["warps"] = int(rng.choice([1, 3, 4, 8, 12, 16]))
    if rng.random() < 0.4:
        kw["stage_bytes"], kw["stages"] = int(rng.choice([1024, 4096, 16384, 32768])), int(rng.choice([2, 3, 5, 9]))
    o = H.opts(**kw) if kw else None
    tau = float(rng.choice([0.1, 0.2, 0.0, 1.0, 0.5]))
    try:
        full = ssd.ssd_verify(view, offd, ids, tau, skip=skip, V=V, opts=o)
    except ssd.SsdError as e:
        assert e.code == ssd.ERR_ARG          # a ring that does not fit: refused on the host
        return
    ee = ssd.ssd_verify_early_exit(view, offd, ids, tau, skip=skip, V=V, opts=o)
    torch.cuda.synchronize()
    assert torch.equal(ee["accepted_len"], full["accepted_len"])
    assert torch.equal(ee["all_accepted"], full["all_accepted"])
    se, sf = H.status_u32(ee["utt_status"]), H.status_u32(full["utt_status"])
    assert not (se & ~sf).any() and not (sf & 0x80000000).any()
    rr = ee["rows_read"].cpu().numpy()
    assert (rr >= 0).all()
    assert (se[rr == lens] == sf[rr == lens]).all()
    al = full["accepted_len"].cpu().numpy()
    sk = skip.cpu().numpy().astype(bool) if skip is not None else np.zeros(B, bool)
    a, c = ee["token_logp"].cpu().numpy(), full["token_logp"].cpu().numpy()
    for b in np.flatnonzero(~sk):
        s = slice(int(off[b]), int(off[b]) + min(int(lens[b]), int(al[b]) + 1))
        fin = np.isfinite(c[s])
        assert np.abs(a[s][fin] - c[s][fin]).max(initial=0.0) <= 2e-5
        np.testing.assert_array_equal(a[s][~fin], c[s][~fin])


@pytest.mark.parametrize("seed", range(40))
def test_frame_statistics_kernels_agree_under_random_options(cuda_device, seed):
    """The bulk-copy kernel under random launch options (grid, warps, lanes per row, where the
    exponentials run) against the plain-load kernel: rows of 1 to 5,000 symbols, ragged batches,
    logits far from zero, views with padded rows."""
    rng = np.random.default_rng(8000 + seed)
    V = int(rng.choice([1, 7, 33, 129, 348, 1025, 4097, 5000]))
    dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
    B = int(rng.choice([1, 3, 17, 64, 300, 2500]))
    T = rng.integers(0, int(rng.choice([5, 40, 400])) + 1, size=B)
    N = int(T.sum())
    if N == 0 or N * V > 1e8:
        T = np.minimum(T, 3) + (np.arange(B) == 0)
        N = int(T.sum())
    dev = cuda_device
    off = torch.from_numpy(np.concatenate([[0], np.cumsum(T)]).astype(np.int64)).to(dev)
    pad = int(rng.integers(0, 9))
    col0 = int(rng.integers(0, pad + 1))
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    shift, scale = float(rng.choice([0.0, 0.0, -150.0, 90.0])), float(rng.choice([0.3, 2.0, 8.0]))
    wide = (torch.randn((N, V + pad), generator=g, device=dev) * scale + shift).to(dtype)
    win = torch.randint(0, V, (N,), generator=g, device=dev)
    wide[torch.arange(N, device=dev), col0 + win] += float(rng.choice([1.0, 6.0, 12.0]))
    view = wide[:, col0:col0 + V]
    blank, cap = int(rng.integers(0, V)), int(rng.choice([1, 50, 200, 600]))
    kw = {}
    if rng.random() < 0.4:
        kw["ctas"] = int(rng.choice([1, 8, 37, 148]))
    if rng.random() < 0.4:
        kw["warps"] = int(rng.choice([1, 2, 5, 8, 12, 16]))
    if rng.random() < 0.4:
        kw["split"] = int(rng.choice([2, 4, 8, 16, 32]))
    if rng.random() < 0.4 and dtype == torch.bfloat16:
        kw["fma_exp"] = int(rng.choice([-1, 1, 2]))
    try:
        a = ssd.ssd_ctc_draft(view, off, blank, cap, V=V, opts=H.opts(**kw) if kw else None)
    except ssd.SsdError as e:
        assert e.code == ssd.ERR_ARG and "split" in kw       # a lane would walk too many chunks
        return
    b = ssd.ssd_ctc_draft(view, off, blank, cap, V=V, opts=H.opts(kernel=1))
    torch.cuda.synchronize()
    for k in ("frame_argmax", "draft_len", "draft_full_len", "utt_status"):
        assert torch.equal(a[k], b[k]), k
    assert not (H.status_u32(a["utt_status"]) != 0).any()
    he, hp = a["frame_entropy"].double(), b["frame_entropy"].double()
    assert float((he - hp).abs().max()) <= H.FLOAT_TOL
    le, lp = a["frame_lse"].double(), b["frame_lse"].double()
    assert float((le - lp).abs().max()) <= H.FLOAT_TOL + 2.5e-7 * float(lp.abs().max())


@pytest.mark.parametrize("seed", range(40))
def test_verify_kernels_agree_under_random_options(cuda_device, seed):
    """ssd_verify's bulk-copy kernel under random launch options (grid, warps, column spans, ring
    shape, exponential split, where rows are finished) against the plain-load kernel, on new
    workspaces that hold whatever the allocator left in them."""
    rng = np.random.default_rng(9000 + seed)
    V = int(rng.choice([1, 9, 257, 1000, 4099, 32000, 50257]))
    dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
    B = int(rng.choice([1, 2, 7, 32, 100, 257, 1000]))
    lens = rng.integers(0, int(rng.choice([1, 3, 10, 60])) + 1, size=B)
    if lens.sum() == 0:
        lens[0] = 2
    while lens.sum() * V > 1e8:
        lens = lens // 2
    M = int(lens.sum())
    if M == 0:
        lens[0] = 1
        M = 1
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    dev = cuda_device
    pad = int(rng.integers(0, 9))
    col0 = int(rng.integers(0, pad + 1))
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    shift, scale = float(rng.choice([0.0, 0.0, -150.0, 90.0])), float(rng.choice([0.3, 2.0, 8.0]))
    wide = (torch.randn((M, V + pad), generator=g, device=dev) * scale + shift).to(dtype)
    ids = torch.randint(0, V, (M,), generator=g, device=dev, dtype=torch.int32)
    keep = torch.rand((M,), generator=g, device=dev) < float(rng.choice([0.5, 0.97, 1.0]))
    rows = torch.arange(M, device=dev)[keep]
    wide[rows, col0 + ids[rows].long()] += float(rng.choice([6.0, 12.0, 30.0]))
    view = wide[:, col0:col0 + V]
    offd = torch.from_numpy(off).to(dev)
    skip = (torch.rand((B,), generator=g, device=dev) < 0.3).to(torch.uint8) if rng.random() < 0.5 else None
    kw = {}
    if rng.random() < 0.3:
        kw["ctas"] = int(rng.choice([1, 8, 37, 148]))
    if rng.random() < 0.3:
        kw["warps"] = int(rng.choice([1, 3, 4, 8, 12, 16]))
    if rng.random() < 0.3:
        kw["split"] = int(rng.choice([1, 2, 3, 7]))
    if rng.random() < 0.3:
        kw["stage_bytes"], kw["stages"] = int(rng.choice([1024, 4096, 16384, 65536])), int(rng.choice([2, 3, 5, 9]))
    if rng.random() < 0.2 and dtype == torch.bfloat16:
        kw["fma_exp"] = int(rng.choice([-1, 1, 2, 3]))
    if rng.random() < 0.3:
        kw["finish"], kw["split"] = 2, 1
    tau = float(rng.choice([0.1, 0.2, 0.5]))
    try:
        a = ssd.ssd_verify(view, offd, ids, tau, skip=skip, V=V, opts=H.opts(**kw) if kw else None)
    except ssd.SsdError as e:
        assert e.code == ssd.ERR_ARG and kw           # a ring that does not fit, finish = 2 on too many utterances
        return
    b = ssd.ssd_verify(view, offd, ids, tau, skip=skip, V=V, opts=H.opts(kernel=1))
    torch.cuda.synchronize()
    sk = skip.cpu().numpy().astype(bool) if skip is not None else np.zeros(B, bool)
    rowmask = torch.from_numpy(np.repeat(~sk, lens)).to(dev)
    la, lb = a["token_logp"].double(), b["token_logp"].double()
    fin = torch.isfinite(lb) & rowmask
    if bool(fin.any()):
        assert float((la[fin] - lb[fin]).abs().max()) <= 5e-5
    if not bool((((lb - np.log(tau)).abs() < H.MARGIN) & rowmask).any()):
        for k in ("accepted_len", "all_accepted", "utt_status"):
            assert torch.equal(a[k], b[k]), k
