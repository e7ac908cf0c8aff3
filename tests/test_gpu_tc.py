"""GPU parity of the tensor-core denoisers (bf16 MLP, large bf16 mixture) against the oracle, which
rounds operands to bfloat16 at the same points. Outputs agree within 2e-2 relative (row L2)."""
import math

import numpy as np
import pytest

import paper_2501_05370_b200 as sds
from paper_2501_05370_b200 import binding as sb
from oracle import sds_oracle as o
import workloads as wl
from helpers import BAND, assert_rows_close, ell_close, oracle_setup, rel_l2

pytestmark = pytest.mark.gpu

TOL = 2e-2


@pytest.mark.parametrize("dims,rows,K", [([128, 256, 128], 300, 7), ([256, 128, 384, 256], 129, 5),
                                         ([128, 128], 64, 3), ([384, 512, 512, 512, 384], 1000, 11)])
def test_mlp_denoiser_rows(dims, rows, K):
    import torch
    w = wl.WORKLOADS["cfg3"].scaled(d=dims[0], B=rows, L=1, K=K, mlp_dims=dims)
    mp = w.mlp_params()
    s = sds.sampler_for(w, mlp=mp)
    den, a, c, sig = oracle_setup(w, mlp=mp)
    rng = np.random.default_rng(3)
    x = rng.standard_normal((rows, dims[0])).astype(np.float32)
    k = rng.integers(0, K, size=rows).astype(np.int32)
    out = s.denoise(torch.from_numpy(x).cuda(), torch.from_numpy(k).cuda()).cpu().numpy()
    assert np.all(np.isfinite(out))
    for r in list(range(0, rows, max(1, rows // 60))) + [rows - 1]:     # the last row of the ragged tile as well
        assert_rows_close(out[r], den(x[r].astype(np.float64), int(k[r])), TOL, r)
    s.close()


@pytest.mark.parametrize("d,ncomp,rows", [(256, 128, 200), (384, 256, 77), (1024, 384, 260),
                                          (4096, 512, 300), (4096, 1024, 515)])   # long K, N % 512 == 0: 256 x 512 logits tiles
def test_large_mixture_denoiser_rows(d, ncomp, rows):
    import torch
    w = wl.WORKLOADS["cfg4"].scaled(d=d, B=rows, L=1, K=50)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    s = sds.sampler_for(w, gmm=gp)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    rng = np.random.default_rng(4)
    x = rng.standard_normal((rows, d)).astype(np.float32)
    x[::5] = 0.7 * gp.means[rng.integers(0, ncomp, size=len(x[::5]))] + 0.3 * x[::5]
    k = rng.integers(0, w.K, size=rows).astype(np.int32)
    out = s.denoise(torch.from_numpy(x).cuda(), torch.from_numpy(k).cuda()).cpu().numpy()
    assert np.all(np.isfinite(out))
    for r in range(0, rows, max(1, rows // 50)):
        assert_rows_close(out[r], den(x[r].astype(np.float64), int(k[r])), TOL, r)
    s.close()


@pytest.mark.parametrize("name,d,ncomp,rows,pattern", [("cfg4", 512, 128, 700, "all"), ("cfg4", 512, 128, 700, "blocks"),
                                                        ("cfg4", 1024, 256, 300, "some"), ("cfg5", 1024, 256, 900, "blocks"),
                                                        ("cfg5", 256, 128, 520, "all"),
                                                        ("cfg5", 256, 128, 76900, "blocks")])   # enough blocks for the lazy plane stores
def test_one_hot_rows_skip_the_mixing_contraction_with_the_same_bits(name, d, ncomp, rows, pattern):
    """Rows that sit next to one component at a low noise level have a single non-zero responsibility.
    Blocks of 256 such rows are not multiplied at all: a copy kernel writes the component's mean (through
    the same affine map). The result must equal the oracle's (2e-2 for the bf16 mixture, 1e-5 for the float
    one) and, bit for bit, what the contraction itself gives (option off). Patterns: every row one-hot;
    whole blocks one-hot next to blocks of broad rows (some tiles skipped, some not, a ragged last block);
    one-hot rows scattered among broad ones (nothing can be skipped)."""
    import torch
    w = wl.WORKLOADS[name].scaled(d=d, B=rows, L=1, K=50)
    gp = w.gmm_params(d=d, ncomp=ncomp)
    s = sds.sampler_for(w, gmm=gp)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    rng = np.random.default_rng(8)
    late = w.K - 2                                           # almost no noise left: alpha close to 1
    k = np.full(rows, late, dtype=np.int32)
    scale = 1.0 if w.sampler == "ula" else math.sqrt(o.ddpm_affine(w.beta())[3][late])
    sharp = (scale * gp.means[rng.integers(0, ncomp, size=rows)] + 0.01 * rng.standard_normal((rows, d))).astype(np.float32)
    ca, cb = rng.integers(0, ncomp, size=rows), rng.integers(0, ncomp - 1, size=rows)
    cb = np.where(cb >= ca, cb + 1, cb)                       # a second, different component
    broad = (scale * 0.5 * (gp.means[ca] + gp.means[cb]) + 1e-4 * rng.standard_normal((rows, d))).astype(np.float32)  # half way: two weights
    x = sharp.copy()
    if pattern == "blocks":
        for blk in range(0, rows, 256):
            if (blk // 256) % 2 == 1:
                x[blk:blk + 256] = broad[blk:blk + 256]
    elif pattern == "some":
        x[::3] = broad[::3]
    xt, kt = torch.from_numpy(x).cuda(), torch.from_numpy(k).cuda()
    got = s.denoise(xt, kt).cpu().numpy()
    ctl = s.get(sb.GET_CTL)
    skipped, ran = int(ctl[10]), int(ctl[8]) + int(ctl[9])
    if pattern == "all":
        assert skipped > 0 and ran == 0
    elif pattern == "blocks":
        assert skipped > 0 and ran > 0
    else:
        assert skipped == 0 and ran > 0
    s.set_option(s.OPT_ONEHOT_ROWS, 0)
    ref = s.denoise(xt, kt).cpu().numpy()
    assert np.array_equal(got, ref)
    tol = TOL if gp.means_bf16 else 1e-5
    is_broad = np.zeros(rows, dtype=bool)
    if pattern == "blocks":
        is_broad[[r for r in range(rows) if (r // 256) % 2 == 1]] = True
    elif pattern == "some":
        is_broad[::3] = True
    for r in list(range(0, rows, max(37, rows // 300))) + [rows - 1]:
        want = den(x[r].astype(np.float64), int(k[r]))
        if w.sampler == "ula" and is_broad[r]:
            # half way between two modes the energy gradient (x - sum r mu)/s^2 is a difference of nearly equal
            # vectors: the error is bounded relative to the size of x, not of the (tiny) result
            assert np.max(np.abs(got[r] - want)) <= 1e-5 * np.sqrt(np.mean(x[r].astype(np.float64) ** 2)) / gp.comp_std ** 2, r
        else:
            assert_rows_close(got[r], want, tol, r)
    s.close()


def _forced_window(s, w, den, seed, off, windows, chains=None, every_position=None, reset=True):
    """Decisions and log ratios of the verify step replayed by the oracle on the GPU's own arrays
    (the denoiser outputs are the GPU's; their parity is checked at 2e-2, row norm and element-wise,
    at the first and last position of every checked chain and at every position of the chains in
    `every_position`). Returns the number of denoiser rows compared."""
    s.set_option(s.OPT_VERIFY_EARLY_EXIT, 0)      # these checks look at every position of the window
    import math
    a32, c32, s32, _ = sds.schedule_for(w)
    a64, c64, s64 = a32.astype(np.float64), c32.astype(np.float64), s32.astype(np.float64)
    B, L, d, K = s.B, s.L, s.d, s.K
    band = tests = den_rows = 0
    if reset:
        s.reset()
    for _ in range(windows):
        ctl = s.get(sb.GET_CTL)
        na = int(ctl[0])
        if na == 0:
            break
        act, rowoff, n = s.get(sb.GET_ACT)[:na], s.get(sb.GET_ROWOFF)[:na + 1], s.get(sb.GET_N)
        Dc = s.get(sb.GET_DC)
        s.draft()
        X, T = s.get(sb.GET_X), s.get(sb.GET_TAIL)
        s.verify_window()
        Dq = s.get(sb.GET_DQ)
        ell, logU, accmask, jstar = s.get(sb.GET_ELL), s.get(sb.GET_LOGU), s.get(sb.GET_ACCMASK), s.get(sb.GET_JSTAR)
        X2, T2 = s.get(sb.GET_X), s.get(sb.GET_TAIL)
        rowk = s.get(sb.GET_ROWK)
        for si, b in enumerate(act):
            if chains is not None and int(b) not in chains:
                continue
            nb = int(n[b]); Lt = min(L, K - nb); r0 = int(rowoff[si])
            W = np.concatenate([X[r0:r0 + Lt], T[b:b + 1]]).astype(np.float64)
            assert np.array_equal(rowk[r0:r0 + Lt], nb + np.arange(Lt))
            full = every_position is not None and int(b) in every_position
            for j in (range(1, Lt + 1) if full else sorted({1, Lt})):
                assert_rows_close(Dq[r0 + j - 1], den(W[j - 1], nb + j - 1), TOL, (int(b), j))
                den_rows += 1
            v = o.verify_window(W, Dq[r0:r0 + Lt], Dc[b], a64, c64, s64, nb, logU[b, :Lt].astype(np.float64))
            amb = np.abs(v["ell"] - logU[b, :Lt]) < BAND
            for j in range(Lt):
                assert ell_close(float(ell[b, j]), float(v["ell"][j]))
                tests += 1
                if amb[j]:
                    band += 1
                else:
                    assert bool((int(accmask[b]) >> j) & 1) == bool(v["acc"][j])
            if not amb.any():
                assert int(jstar[b]) == v["jstar"]
                js = int(jstar[b])
                if js <= Lt:
                    assert_rows_close(X2[r0 + js] if js < Lt else T2[b], v["Y_reflect"], 1e-5, (int(b), js))
        s.advance()
    assert band <= max(2, 2e-3 * tests)
    return den_rows


def test_mlp_window_forced_and_free_run():
    dims = [256, 384, 384, 256]
    w = wl.WORKLOADS["cfg3"].scaled(d=256, B=70, L=8, K=40, mlp_dims=dims)
    mp = w.mlp_params()
    s = sds.sampler_for(w, mlp=mp, seed=31, chain_id_offset=7)
    den, a, c, sig = oracle_setup(w, mlp=mp)
    _forced_window(s, w, den, 31, 7, 4)
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(out)) and np.array_equal(s.get(sb.GET_N), np.full(70, 40))
    assert np.all(calls >= 1 + 40 // 8) and np.all(calls <= 41)
    out2 = s.sample_all()[0].cpu().numpy()
    assert np.array_equal(out, out2)                     # deterministic
    s.close()


def test_large_mixture_window_forced_and_free_run():
    w = wl.WORKLOADS["cfg4"].scaled(d=512, B=40, L=16, K=60)
    gp = w.gmm_params(d=512, ncomp=128)
    s = sds.sampler_for(w, gmm=gp, seed=41)
    den, a, c, sig = oracle_setup(w, gmm=gp)
    _forced_window(s, w, den, 41, 0, 3)
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(out)) and np.array_equal(s.get(sb.GET_N), np.full(40, 60))
    # statistical agreement of the free run with the oracle's speculative chain (bf16 denoiser:
    # trajectories are compared in law, not bit by bit): mean number of target calls
    oc = [o.speculative_chain(den, a, c, sig, w.L, 41, b, w.d)["nfe_calls"] for b in range(12)]
    assert abs(np.mean(oc) - calls.mean()) <= 4 * (np.std(oc) / np.sqrt(12) + calls.std() / np.sqrt(40)) + 1.0
    s.close()


@pytest.mark.parametrize("name", ["cfg3", "cfg4"])
def test_full_size_tensor_core_windows_on_sampled_chains(name):
    """Full benchmark sizes and launch shapes (thousands of GEMM tiles). The oracle replays sixteen
    chains: the first window (every chain at step 0, full row count), then, after forty more windows,
    a window in which the chains sit at different steps, some of them so close to the end that their
    windows are shorter than L and one already finished, so that the row count is no multiple of the
    tile height and the last tile of every GEMM is ragged; there every position of the sixteen chains
    is compared with the oracle's denoiser (the first window: every position of four of them).
    Then the whole run: every chain ends at n = K with finite state and consistent counters."""
    import torch
    w = wl.WORKLOADS[name]
    if name == "cfg3":
        mp_ = w.mlp_params()
        s = sds.sampler_for(w, mlp=mp_)
        den, a, c, sig = oracle_setup(w, mlp=mp_)
    else:
        gp = w.gmm_params()
        s = sds.sampler_for(w, gmm=gp)
        den, a, c, sig = oracle_setup(w, gmm=gp)
    rng = np.random.default_rng(11)
    chains = sorted({0, 1, 2, 3, w.B // 2 + 1, w.B - 2, w.B - 1} | set(int(x) for x in rng.choice(w.B, size=9, replace=False)))
    chains = chains[:16] if len(chains) > 16 else chains
    first = _forced_window(s, w, den, w.sample_seed, 0, 1, chains=set(chains), every_position=set(chains[:4]))
    assert first >= 4 * w.L
    for _ in range(40):
        s.draft(); s.verify_window(); s.advance(sync=False)
    n = s.get(sb.GET_N).copy()
    assert len(set(n[chains].tolist())) > 1                   # the chains have spread over the steps
    n[chains[1]] = w.K - 3                                    # a window of three positions
    n[chains[2]] = w.K                                        # a finished chain: no rows at all
    n[chains[3]] = w.K - 1                                    # a window of one position
    n[chains[-1]] = w.K - (w.L - 1)                           # the last chain: one position short of a full window
    if int(np.minimum(w.L, w.K - n)[n < w.K].sum()) % 128 == 0:
        n[chains[4]] = w.K - 2
    s.set_state(n=torch.from_numpy(n).cuda())
    ctl = s.get(sb.GET_CTL)
    assert int(ctl[0]) == int(np.sum(n < w.K)) and int(ctl[1]) == int(np.minimum(w.L, w.K - n)[n < w.K].sum())
    assert int(ctl[1]) % 128 != 0                             # ragged: the row count is no multiple of a tile
    late = _forced_window(s, w, den, w.sample_seed, 0, 1, chains=set(chains), every_position=set(chains), reset=False)
    assert late >= 11 * w.L
    out, calls, rows = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(out)) and np.array_equal(s.get(sb.GET_N), np.full(w.B, w.K))
    assert np.all(calls >= 1 + -(-w.K // w.L)) and np.all(calls <= 1 + w.K)
    assert np.all(rows >= w.K + 1) and np.all(rows <= 1 + (calls - 1) * w.L)
    s.close()


def test_bounded_wait_runs_out_and_reports():
    """A wait on a barrier that nothing completes gives up after its poll limit and says so; the
    context stays usable (the next kernel runs)."""
    import torch
    st = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    rc = sb.load().sds_selftest_bounded_wait(2000, st.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == sb.SDS_OK
    torch.cuda.synchronize()
    assert int(st.item()) == 1
    assert float((torch.ones(4, device="cuda") * 2).sum().item()) == 8.0


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_runs_agree_bitwise_across_kernel_options(name):
    """At the benchmark sizes: the verify kernel that exits early, advances its chains and draws the
    drafted states again instead of reading them, the CTA-pair GEMM, the mixing GEMM that leaves blocks
    of one-hot rows to a copy kernel and the whole-chain kernel change how the work is done, not one bit
    of the result, and a repeated run reproduces itself."""
    import torch
    w = wl.WORKLOADS[name]
    s = sds.sampler_for(w)
    ref = None
    for fuse, early, pair, whole, raw, regen, hot in [(1, 1, 1, 1, 1, 1, 1), (1, 1, 1, 1, 1, 1, 1), (1, 1, 1, 1, 1, 0, 1), (0, 1, 1, 1, 1, 1, 1),
                                                     (1, 0, 1, 1, 1, 1, 1), (1, 1, 1, 1, 0, 1, 1), (1, 1, 1, 1, 1, 1, 0), (1, 1, 0, 1, 0, 1, 1), (1, 1, 1, 1, 1, 2, 1),
                                                     (0, 0, 0, 0, 0, 0, 0)]:
        s.set_option(s.OPT_FUSE_ADVANCE, fuse); s.set_option(s.OPT_VERIFY_EARLY_EXIT, early)
        s.set_option(s.OPT_GEMM_PAIR, pair); s.set_option(s.OPT_WHOLE_CHAIN_KERNEL, whole)
        s.set_option(s.OPT_RAW_ROWS, raw); s.set_option(s.OPT_REGEN_DRAFTS, regen); s.set_option(s.OPT_ONEHOT_ROWS, hot)
        got = [x.clone() for x in s.sample_all()]
        if ref is None:
            ref = got
            assert torch.isfinite(ref[0]).all()
        else:
            assert all(torch.equal(a, b) for a, b in zip(ref, got)), (fuse, early, pair, whole, raw, regen, hot)
    s.close()


@pytest.mark.parametrize("kind,d,L,B", [("gmm", 512, 9, 21), ("gmm", 1536, 7, 13), ("mlp", 3072, 8, 10), ("gmm", 4096, 6, 9),
                                         ("mlp", 8192, 5, 5), ("gmm", 16384, 6, 4), ("gmm", 512, 1, 5), ("gmm", 1024, 2, 7),
                                         ("gmm", 2048, 32, 3), ("gmm", 12416, 5, 5), ("gmm", 6272, 4, 5)])
def test_drafted_states_drawn_again_give_the_same_bits(kind, d, L, B):
    """Targets that read only the bf16 rows (the MLP, the bf16 mixture): inside sds_sample_all the draft
    kernel stores only those rows and verify runs the draft recurrence again from Y_n, the carried
    output and the chain's noise. One case per verify kernel shape; windows whose first rejection
    falls at every offset of a block of positions, windows that accept everything, a ragged last
    window. Same bits as with the rows read back, as with the advance kernel, and as the step-wise calls."""
    K = 3 * L + 4
    if kind == "mlp":
        w = wl.WORKLOADS["cfg3"].scaled(d=d, B=B, L=L, K=K, mlp_dims=[d, 256, d])
        s = sds.sampler_for(w, mlp=w.mlp_params(), seed=81)
    else:
        w = wl.WORKLOADS["cfg4"].scaled(d=d, B=B, L=L, K=K)
        s = sds.sampler_for(w, gmm=w.gmm_params(d=d, ncomp=128), seed=81)
    s.set_option(s.OPT_REGEN_DRAFTS, 2)                   # in every window
    got = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(got[0]))
    ctl = s.get(sb.GET_CTL)
    windows = int(ctl[2])
    assert int(ctl[13]) == int(ctl[12]) > 0 and int(ctl[14]) == 0      # every position verified on states made again, no float rows
    s.set_option(s.OPT_REGEN_DRAFTS, 1)                   # window by window, from the positions the last window needed
    mixed = [x.cpu().numpy() for x in s.sample_all()]
    assert all(np.array_equal(x, y) for x, y in zip(got, mixed))
    assert int(s.get(sb.GET_CTL)[12]) == int(ctl[12])     # the same positions were evaluated
    s.set_option(s.OPT_REGEN_DRAFTS, 0)
    back = [x.cpu().numpy() for x in s.sample_all()]
    assert int(s.get(sb.GET_CTL)[13]) == 0
    assert all(np.array_equal(x, y) for x, y in zip(got, back))
    assert windows == int(s.get(sb.GET_CTL)[2])
    s.set_option(s.OPT_FUSE_ADVANCE, 0)
    sep = [x.cpu().numpy() for x in s.sample_all()]
    assert all(np.array_equal(x, y) for x, y in zip(got, sep))
    s.reset()
    na, advs = B, []
    while na > 0:
        n0 = s.get(sb.GET_N).copy()
        s.draft(); s.verify_window(); na = s.advance()
        advs.append(s.get(sb.GET_N) - n0)
    assert np.array_equal(s.get(sb.GET_Y), got[0])
    assert np.array_equal(s.get(sb.GET_NFE_CALLS), got[1]) and np.array_equal(s.get(sb.GET_NFE_ROWS), got[2])
    adv = np.concatenate(advs)
    if kind == "gmm" and L >= 5:                          # (the random network's drafts are rejected at once)
        assert len(set(adv[adv > 0].tolist())) >= 3       # the windows did end at several different positions
    s.close()


@pytest.mark.parametrize("kind,d,L,B", [("gmm", 1536, 7, 13), ("mlp", 3072, 8, 10), ("gmm", 16384, 6, 4), ("gmm", 2048, 32, 3)])
def test_staged_windows_on_the_tensor_core_targets(kind, d, L, B):
    """Staged windows with the bf16 targets: states drafted again or read back, one-hot rows read from the means
    table, every stage length: the final states of whole windows, bit for bit."""
    K = 3 * L + 4
    if kind == "mlp":
        w = wl.WORKLOADS["cfg3"].scaled(d=d, B=B, L=L, K=K, mlp_dims=[d, 256, d])
        s = sds.sampler_for(w, mlp=w.mlp_params(), seed=83)
    else:
        w = wl.WORKLOADS["cfg4"].scaled(d=d, B=B, L=L, K=K)
        s = sds.sampler_for(w, gmm=w.gmm_params(d=d, ncomp=128), seed=83)
    ref = [x.cpu().numpy() for x in s.sample_all()]
    assert np.all(np.isfinite(ref[0]))
    for regen in (1, 2, 0):
        s.set_option(s.OPT_REGEN_DRAFTS, regen)
        for stage in (1, 2, 3, L, s.STAGED_ADAPTIVE):
            s.set_option(s.OPT_STAGED_WINDOWS, stage)
            got = [x.cpu().numpy() for x in s.sample_all()]
            assert np.array_equal(got[0], ref[0]), (regen, stage)
            assert np.all(got[2] <= ref[2]) and np.all(got[1] >= ref[1]), (regen, stage)
            if stage == L:
                assert np.array_equal(got[1], ref[1]) and np.array_equal(got[2], ref[2])
    s.close()


@pytest.mark.parametrize("name", ["cfg3", "cfg4"])
def test_full_size_staged_run_gives_the_samples_of_whole_windows(name):
    """The bench configurations at full size, stage length chosen by the library: final states bit for bit those
    of whole windows, fewer target rows, and the counters add up (every chain took K steps)."""
    import torch
    w = wl.WORKLOADS[name]
    s = sds.sampler_for(w, **({"mlp": w.mlp_params()} if w.denoiser == "mlp" else {"gmm": w.gmm_params()}), seed=w.sample_seed)
    ref = [x.clone() for x in s.sample_all()]
    s.set_option(s.OPT_STAGED_WINDOWS, s.STAGED_ADAPTIVE)
    got = s.sample_all()
    assert torch.equal(got[0], ref[0])
    assert int(got[2].sum()) < int(ref[2].sum()) and int(got[1].sum()) >= int(ref[1].sum())
    assert np.array_equal(s.get(sb.GET_N), np.full(w.B, w.K))
    assert int(s.get(sb.GET_CTL)[7]) > 0
    s.close()
