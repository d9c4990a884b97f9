"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded
inputs.  Bit-exact on symbols, residuals, histograms, headers, code tables, bitstreams, side
information and averaged gradients; GenNorm fit parameters within 1e-5 relative."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

FORMATS = [(1, 2), (3, 2), (4, 3)]


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2203_09044_b200 import binding as b
    b.lib()          # raises if the CUDA library is not built: there is no fallback
    return b


def _bits(x):
    return np.ascontiguousarray(x).view(np.uint32)


def compare_iteration(b, plan, out, r, m_gpu, m_cpu, tag=""):
    """One encoded iteration: everything co3_encode produced vs the oracle's IterationResult."""
    U, d = plan.U, plan.d
    if plan.bias_mode != b.CODE_LAGGED:          # that mode keeps no symbols: the bit-exact payload stands for them
        sym = plan.debug_symbols().cpu().numpy()
        assert np.array_equal(sym, r.sym), f"{tag} symbols"
    assert np.array_equal(_bits(m_gpu.cpu().numpy()[:, :d]), _bits(m_cpu[:, :d])), f"{tag} residual"
    assert np.array_equal(plan.debug_hist(), r.hist), f"{tag} histogram"
    for l in range(plan.S):
        beta, alpha, N, S1, S2 = plan.get_fit(l)
        assert N == r.moments[l, 0], f"{tag} N"
        np.testing.assert_allclose([S1, S2], r.moments[l, 1:], rtol=1e-12, err_msg=f"{tag} moments")
        np.testing.assert_allclose([beta, alpha], r.fit[l], rtol=1e-5, err_msg=f"{tag} fit")
    hdr = b.hdr_to_numpy(out["hdr"])
    assert np.array_equal(hdr, r.hdr), f"{tag} header {hdr[hdr != r.hdr]} vs {r.hdr[hdr != r.hdr]}"
    if plan.bias_mode == b.CODE_EMPIRICAL:          # the code is the length table the encoder wrote
        assert np.array_equal(out["code_lens"].cpu().numpy(), r.lens), f"{tag} code lengths (side information)"
    else:
        lens, codes = plan.debug_code(out["hdr"])
        assert np.array_equal(lens, r.lens), f"{tag} code lengths"
        assert np.array_equal(codes, r.codes), f"{tag} codewords"
    co = out["chunk_off"].cpu().numpy().view(np.uint32)
    assert np.array_equal(co, r.chunk_off), f"{tag} chunk offsets"
    assert np.array_equal(out["sub_bits"].cpu().numpy().view(np.uint16)[:, :plan.n_sub],
                          r.sub_bits[:, :plan.n_sub]), f"{tag} sub_bits"
    assert np.array_equal(out["user_bits"].cpu().numpy().view(np.uint64), r.user_bits), f"{tag} user_bits"
    pay = out["bitstream"].cpu().numpy().view(np.uint32)
    for u in range(U):
        n = int(co[u, -1])
        if n <= plan.cap_words:
            assert np.array_equal(pay[u, :n], r.payload[u, :n]), f"{tag} bitstream user {u}"


def run_case(b, oracle, d, U, E, M, off, grads, gamma=0.9, mode=1, cap=None, decode_plan=None, rule=0):
    """grads: list of [U][ld] float32 cuda tensors, one per iteration (ld is taken from them)."""
    plan = b.Plan(d, U, E, M, off, gamma=gamma, bias_mode=mode, cap_words=cap, ld=int(grads[0].shape[1]),
                  bias_rule=rule)
    orc = oracle.OracleCO3(d, U, E, M, off, gamma=gamma, mode=mode, cap_words=plan.cap_words, rule=rule)
    assert plan.worst_case_words == orc.worst_case_words
    assert (plan.n_chunks, plan.n_sub) == (orc.part.n_chunks, orc.part.n_sub)
    out = plan.alloc_outputs()
    m_gpu = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
    m_cpu = np.zeros((U, plan.ld), np.float32)
    dec = decode_plan or plan
    results = []
    for t, g in enumerate(grads):
        g_cpu = g.cpu().numpy()
        plan.encode(g, m_gpu, out)
        r = orc.encode(g_cpu, m_cpu)
        compare_iteration(b, plan, out, r, m_gpu, m_cpu, tag=f"t={t}")
        flags, nf = plan.status()
        assert nf == r.nonfinite or t > 0
        if r.status == oracle.OK:
            avg = dec.decode_aggregate(out).cpu().numpy()
            rc, avg_o, _ = orc.decode_aggregate(r.payload, r.sub_bits, r.chunk_off, r.hdr,
                                                lens=r.lens if mode == 3 else None)
            assert rc == oracle.OK
            assert np.array_equal(_bits(avg), _bits(avg_o)), f"t={t} averaged gradient"
            assert not (dec.status()[0] & b.FLAG_CORRUPT)
        results.append((r, flags))
    return plan, orc, out, results


def _grads(wl, iters, device="cuda"):
    return [wl.gradient(t, device=device).to("cuda") for t in range(iters)]


# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_configs_scaled_down(binding, oracle, idx):
    """The four benchmark configurations at a size the oracle finishes in seconds: several
    tiles, ragged tails, all their segments/users/formats, error feedback over iterations."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(idx, d={0: 70_001, 1: 200_000, 2: 150_010, 3: 300_007}[idx])
    run_case(binding, oracle, wl.d, wl.n_users, wl.exp_bits, wl.mant_bits, wl.seg_offsets,
             _grads(wl, 4), gamma=wl.gamma)


def test_padded_rows_as_the_benchmark_lays_them_out(binding, oracle):
    """Rows that start on 16 KiB boundaries (row stride > d): the padding between users is never
    read as data nor written."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=90_000, n_users=3).align_rows()
    assert wl.ld % 4096 == 0 and wl.ld > wl.d
    grads = _grads(wl, 3)
    for g in grads:
        g[:, wl.d:] = 7.0                         # poison: must not leak into moments, symbols or residual
    plan, orc, out, res = run_case(binding, oracle, wl.d, wl.n_users, 4, 3, wl.seg_offsets, grads, gamma=wl.gamma)


@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("U", [1, 2, 3, 5, 8, 9, 16])
def test_users_and_formats(binding, oracle, E, M, U):
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(20_000 + 37 * U, U, 1.0, E, M)
    run_case(binding, oracle, wl.d, U, E, M, wl.seg_offsets, _grads(wl, 2, "cpu"))


@pytest.mark.parametrize("beta", [0.5, 1.0, 2.0])
def test_shapes_fp4(binding, oracle, beta):
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 16, 8, beta, 1, 2)
    run_case(binding, oracle, wl.d, 8, 1, 2, wl.seg_offsets, _grads(wl, 3, "cpu"))


@pytest.mark.parametrize("gamma", [0.0, 1.0])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_gamma_and_bias_modes(binding, oracle, gamma, mode):
    gen = torch.Generator().manual_seed(5)
    d, U = 30_001, 3
    ld = (d + 3) // 4 * 4
    grads = []
    for t in range(4):                                   # scale drifts: the modes differ for t >= 1
        g = torch.zeros((U, ld))
        g[:, :d] = torch.randn((U, d), generator=gen) * (1e-3 * 3.0 ** t)
        grads.append(g.cuda())
    run_case(binding, oracle, d, U, 3, 2, [0, 12_345, d], grads, gamma=gamma, mode=mode)


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("E,M", FORMATS)
def test_l2_optimal_bias_rule(binding, oracle, E, M, mode):
    """CO3_RULE_OPT (the integer bias of least expected squared error for the plan's own format
    instead of the paper's polynomial): bit-exact against the oracle's rule in every mode, on layers
    of different shapes and drifting scales; for the 6- and 8-bit formats, for which the polynomial
    was not made, it does change the bias."""
    from paper_2203_09044_b200 import inputs
    gen = torch.Generator().manual_seed(77 + E)
    d, U, off = 40_000, 3, [0, 9_000, 22_222, 40_000]
    grads = []
    for t in range(3):
        g = torch.zeros((U, d))
        for l, beta in enumerate((0.5, 1.0, 2.0)):
            n = off[l + 1] - off[l]
            for u in range(U):
                g[u, off[l]:off[l + 1]] = inputs.gennorm(n, beta, 1e-3 * 2.5 ** t * (l + 1), gen)
        grads.append(g.cuda())
    plan, orc, out, res = run_case(binding, oracle, d, U, E, M, off, grads, mode=mode, rule=1)
    poly = oracle.OracleCO3(d, U, E, M, off, mode=mode, rule=0)
    r0 = poly.encode(grads[0].cpu().numpy(), np.zeros((U, d), np.float32))
    if (E, M) != (1, 2):
        assert not np.array_equal(r0.bias, res[0][0].bias)


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_fully_lagged_code_configs_scaled_down(binding, oracle, idx):
    """Convert and pack in one pass (header fixed by the previous iteration): the four benchmark
    configurations scaled down, several iterations, everything bit-exact against the oracle's
    LAGGED_CODE mode."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(idx, d={0: 70_001, 1: 200_000, 2: 150_010, 3: 300_007}[idx])
    run_case(binding, oracle, wl.d, wl.n_users, wl.exp_bits, wl.mant_bits, wl.seg_offsets,
             _grads(wl, 4), gamma=wl.gamma, mode=2)


def test_fully_lagged_code_ragged_and_fp4(binding, oracle):
    gen = torch.Generator().manual_seed(16)
    for d, off, U, E, M in ((1, [0, 1], 1, 4, 3), (4097, [0, 4097], 2, 1, 2), (10_000, [0, 1, 130, 4096, 4097, 9_999, 10_000], 3, 1, 2),
                            (33_333, [0, 7, 8, 20_000, 33_333], 9, 3, 2)):
        ld = (d + 3) // 4 * 4
        grads = []
        for t in range(3):
            g = torch.zeros((U, ld))
            g[:, :d] = torch.randn((U, d), generator=gen) * 1e-2
            grads.append(g.cuda())
        run_case(binding, oracle, d, U, E, M, off, grads, mode=2)


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_empirical_histogram_code_configs_scaled_down(binding, oracle, idx):
    """CO3_CODE_EMPIRICAL: per-iteration Huffman codes from the symbol histogram, built on the device,
    length tables as side information; everything bit-exact against the oracle's mode, and the
    decoder needs nothing but the stream, the header's bias and that table."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(idx, d={0: 70_001, 1: 200_000, 2: 150_010, 3: 300_007}[idx])
    plan, orc, out, res = run_case(binding, oracle, wl.d, wl.n_users, wl.exp_bits, wl.mant_bits, wl.seg_offsets,
                                   _grads(wl, 3), gamma=wl.gamma, mode=3)
    # a second plan that never encoded decodes the stream from its side information alone
    dec = binding.Plan(wl.d, wl.n_users, wl.exp_bits, wl.mant_bits, wl.seg_offsets, bias_mode=3)
    avg1 = plan.decode_aggregate(out).cpu().numpy()
    avg2 = dec.decode_aggregate(out, avg=torch.zeros(wl.d, device="cuda")).cpu().numpy()
    assert np.array_equal(_bits(avg1), _bits(avg2)) and dec.status()[0] == 0
    # a length table that is not a complete prefix code is reported, never followed out of bounds
    bad = dict(out)
    bad["code_lens"] = out["code_lens"].clone()
    bad["code_lens"][0, 1] = 0
    dec.decode_aggregate(bad, avg=torch.zeros(wl.d, device="cuda"))
    assert dec.status(clear=True)[0] & binding.FLAG_CORRUPT
    bad["code_lens"] = out["code_lens"].clone()
    bad["code_lens"][0, 2:5] = 1                    # three one-bit codewords: oversubscribed
    dec.decode_aggregate(bad, avg=torch.zeros(wl.d, device="cuda"))
    assert dec.status(clear=True)[0] & binding.FLAG_CORRUPT


@pytest.mark.slow
def test_empirical_histogram_code_needs_large_weight_floors(binding, oracle):
    """A heavy-tailed layer of 67 million symbols: the unrestricted Huffman tree of its counts is far
    deeper than 16, and the weight floor that limits it lies above 2^9 (the largest floor the model
    codes ever need), so the device must try the same floors as the oracle, up to 2^31."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(3, d=1 << 24, n_users=4)
    plan, orc, out, res = run_case(binding, oracle, wl.d, 4, 4, 3, wl.seg_offsets, _grads(wl, 1), mode=3)
    assert int(res[0][0].floor[0]) > 512


def test_empirical_histogram_code_ragged_fp4_many_users(binding, oracle):
    gen = torch.Generator().manual_seed(26)
    for d, off, U, E, M in ((1, [0, 1], 1, 4, 3), (10_000, [0, 1, 130, 4096, 4097, 9_999, 10_000], 3, 1, 2),
                            (33_333, [0, 7, 8, 20_000, 33_333], 9, 3, 2)):
        ld = (d + 3) // 4 * 4
        grads = []
        for t in range(2):
            g = torch.zeros((U, ld))
            g[:, :d] = torch.randn((U, d), generator=gen) * 1e-2
            grads.append(g.cuda())
        run_case(binding, oracle, d, U, E, M, off, grads, mode=3)


def test_ragged_segments_and_tiny_inputs(binding, oracle):
    gen = torch.Generator().manual_seed(6)
    for d, off in ((1, [0, 1]), (5, [0, 2, 2, 5]), (130, [0, 1, 130]), (4097, [0, 4096, 4097]),
                   (9000, [0, 5, 5, 4101, 8192, 9000]), (12_289, [0, 3, 127, 128, 129, 4095, 4097, 12_289])):
        ld = (d + 3) // 4 * 4
        grads = []
        for t in range(2):
            g = torch.zeros((2, ld))
            g[:, :d] = torch.randn((2, d), generator=gen) * 1e-2
            grads.append(g.cuda())
        run_case(binding, oracle, d, 2, 4, 3, off, grads)


@pytest.mark.parametrize("seed", range(40))
def test_random_plans(binding, oracle, seed):
    """Plans drawn at random: size, segment cuts (tiny, empty and chunk-straddling layers), user count,
    format, bias mode and rule, memory weight, row padding, per-layer scales spread over ten binades,
    a few exact zeros and large outliers, layers whose scale jumps or vanishes between iterations.  Three
    iterations each, everything compared."""
    rng = np.random.default_rng(9000 + seed)
    d = int(rng.choice([rng.integers(1, 300), rng.integers(300, 9000), rng.integers(9000, 70_000)]))
    U = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 12, 16, 17, 33]))
    E, M = FORMATS[int(rng.integers(0, 3))]
    mode = int(rng.choice([0, 1, 1, 2, 3]))
    rule = int(rng.integers(0, 2))
    gamma = float(rng.choice([0.0, 0.5, 0.9, 1.0]))
    n_cut = int(rng.integers(0, min(12, d)))
    cuts = np.sort(rng.integers(0, d + 1, size=n_cut))               # repeated cuts = empty layers
    if n_cut and rng.random() < 0.5:
        cuts[rng.integers(0, n_cut)] = min(d, 4096 * int(rng.integers(0, d // 4096 + 1)))   # a cut on the chunk grid
        cuts = np.sort(cuts)
    off = [0] + [int(c) for c in cuts] + [d]
    ld = (d + 3) // 4 * 4 + 4 * int(rng.integers(0, 3)) * int(rng.integers(0, 40))
    gen = torch.Generator().manual_seed(9000 + seed)
    scales = torch.tensor(np.exp2(rng.uniform(-16, -6, size=len(off) - 1)), dtype=torch.float32)
    grads = []
    for t in range(3):
        g = torch.zeros((U, ld))
        x = torch.randn((U, d), generator=gen)
        for l in range(len(off) - 1):                    # (a layer's scale now and then jumps by 32 either way, or to zero)
            x[:, off[l]:off[l + 1]] *= scales[l] * (1.0 + 0.3 * t) * float(rng.choice([1.0, 1.0, 1.0, 32.0, 1.0 / 32.0, 0.0]))
        x[torch.rand((U, d), generator=gen) < 0.01] = 0.0
        x[torch.rand((U, d), generator=gen) < 0.002] *= 300.0
        g[:, :d] = x
        grads.append(g.cuda())
    run_case(binding, oracle, d, U, E, M, off, grads, gamma=gamma, mode=mode, rule=rule)


def _scaled_grads(U, d, ld, off, scales_per_iter, seed, far=None, neg_zero=False):
    """Gaussian gradients whose scale changes from iteration to iteration (scales_per_iter[t][layer]);
    far = (layer, count, value): that many elements of the layer set to +-value in every ODD iteration (so
    that they arrive under a bias that was fitted without them)."""
    gen = torch.Generator().manual_seed(seed)
    grads = []
    for t, sc in enumerate(scales_per_iter):
        g = torch.zeros((U, ld))
        x = torch.randn((U, d), generator=gen)
        for l in range(len(off) - 1):
            x[:, off[l]:off[l + 1]] *= sc[l]
        if far is not None and t % 2 == 1:
            l, count, value = far
            idx = torch.randint(off[l], off[l + 1], (U, count), generator=gen)
            sign = torch.where(torch.rand((U, count), generator=gen) < 0.5, -1.0, 1.0)
            x.scatter_(1, idx, sign * value)
        if neg_zero:
            x[:, ::7] = -0.0
        g[:, :d] = x
        grads.append(g.cuda())
    return grads


@pytest.mark.parametrize("E,M", FORMATS)
def test_current_bias_when_the_guess_is_wrong(binding, oracle, E, M):
    """Bias from the current moments, t >= 1: the convert pass runs under the previous iteration's bias and
    the layers whose bias comes out different are converted again from what was stored.  Here every
    layer's scale jumps by factors of 4 to 64 between iterations, so every guess is wrong: large layers
    (the re-conversion pass), small ones (the fit's own block), a layer of one element, an empty one,
    chunk-straddling ones; exact zeros of both signs ride along."""
    d, U = 70_000, 3
    off = [0, 1, 65, 65, 5000, 9000, 30_000, 30_100, d]
    ld = (d + 3) // 4 * 4 + 8
    L = len(off) - 1
    scales = [[1e-3 * 4.0 ** ((t * (l + 1)) % 4) for l in range(L)] for t in range(5)]
    grads = _scaled_grads(U, d, ld, off, scales, seed=77, neg_zero=True)
    for gamma in (0.0, 0.9):
        plan, orc, out, res = run_case(binding, oracle, d, U, E, M, off, grads, gamma=gamma, mode=0)
        biases = np.stack([r.hdr[:, 0] for r, _ in res])
        assert (np.diff(biases, axis=0) != 0).sum() >= 2 * (L - 1), "the biases were meant to move"
        assert plan.status()[0] == 0


def test_current_bias_with_elements_far_beyond_the_format(binding, oracle):
    """Elements some 2^20 times the largest grid value cannot be rebuilt from symbol and memory (their
    residual is rounded); the convert pass keeps them on a side list and the re-conversion takes them
    from there.  NaN and Inf in the same layers."""
    d, U = 40_000, 2
    off = [0, 100, 20_000, d]
    ld = d
    scales = [[1e-3, 1e-3, 1e-3 * 16.0 ** (t % 2)] for t in range(4)]
    for layer in (0, 1):                                   # a small layer (the fit's block) and a large one (the pass)
        grads = _scaled_grads(U, d, ld, off, scales, seed=78 + layer, far=(layer, 40, 3e9))
        for g in grads:
            g[0, off[layer] + 3] = float("nan")
            g[1, off[layer] + 5] = float("-inf")
        plan, orc, out, res = run_case(binding, oracle, d, U, 4, 3, off, grads, gamma=0.9, mode=0)
        flags = plan.status()[0]
        assert flags & binding.FLAG_NONFINITE and not (flags & binding.FLAG_INEXACT)


def test_current_bias_after_layers_of_zeros_and_of_tiny_values(binding, oracle):
    """A layer that is all zeros (its bias is the lowest one) and then is not, a layer whose scale jumps
    by 10^27 (every element lies far beyond what the previous bias could hold: thousands of side-list
    entries), and back; next to a steady layer."""
    d, U = 30_000, 3
    off = [0, 5000, 10_000, 20_000, d]
    scales = [[0.0, 1e-30, 1e-3, 1e-3], [0.0, 1e-3, 1e-3, 0.0], [1e-3, 1e-30, 1e-3, 0.0], [0.0, 3e-2, 1e-3, 1e-4],
              [2e-3, 1e-3, 1e-3, 0.0]]
    for E, M in ((4, 3), (1, 2)):
        grads = _scaled_grads(U, d, d, off, scales, seed=81)
        plan, orc, out, res = run_case(binding, oracle, d, U, E, M, off, grads, gamma=0.5, mode=0)
        assert plan.status()[0] == 0


def test_current_bias_side_list_overflow_is_reported(binding):
    """More far-out elements in one iteration than the side list holds (in a layer whose bias they change):
    CO3_FLAG_INEXACT.  With fewer of them than the list holds nothing is raised."""
    b = binding
    d, U = 120_000, 2
    off = [0, 30_000, d]
    for moving, count in ((False, 1500), (True, 80_000)):
        scales = [[1e-3, 1e-3] for t in range(3)]
        grads = _scaled_grads(U, d, d, off, scales, seed=80, far=(1, count, 3e9))
        plan = b.Plan(d, U, 4, 3, off, gamma=0.0, bias_mode=b.BIAS_CURRENT)
        out = plan.alloc_outputs()
        m = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
        for g in grads:
            plan.encode(g, m, out)
        flags = plan.status()[0]
        assert bool(flags & b.FLAG_INEXACT) == moving, (moving, flags)
        plan.close()


def test_current_bias_two_implementations_agree(binding, monkeypatch):
    """CO3_TWO_PASS=1 keeps the statistics pass in every iteration (Algorithm 1 line 8 in its printed order);
    the default runs it at t = 0 only and repairs wrong guesses.  Same bits."""
    b = binding
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=400_000, n_users=4)
    outs = []
    for two_pass in ("0", "1"):
        monkeypatch.setenv("CO3_TWO_PASS", two_pass)
        plan = b.Plan(wl.d, wl.n_users, 4, 3, wl.seg_offsets, gamma=wl.gamma, bias_mode=b.BIAS_CURRENT, ld=wl.ld)
        out = plan.alloc_outputs()
        m = torch.zeros((wl.n_users, plan.ld), dtype=torch.float32, device="cuda")
        rec = []
        for t in range(5):
            g = wl.gradient(t, device="cuda") * (1.0 if t % 2 == 0 else 5.0)
            plan.encode(g, m, out)
            n = out["chunk_off"][:, -1].cpu().numpy()
            rec.append((out["hdr"].clone(), out["chunk_off"].clone(), m.clone(), plan.debug_symbols().clone(),
                        [out["bitstream"][u, :int(n[u])].clone() for u in range(wl.n_users)], plan.debug_hist().copy(),
                        plan.decode_aggregate(out).clone()))
        assert plan.status()[0] == 0
        outs.append(rec)
        plan.close()
    for t, (x, y) in enumerate(zip(*outs)):
        assert torch.equal(x[0], y[0]) and torch.equal(x[1], y[1]), f"t={t} header / offsets"
        assert torch.equal(x[2].view(torch.int32), y[2].view(torch.int32)), f"t={t} residual"
        assert torch.equal(x[3], y[3]), f"t={t} symbols"
        assert all(torch.equal(p, q) for p, q in zip(x[4], y[4])), f"t={t} payload"
        assert np.array_equal(x[5], y[5]), f"t={t} histogram"
        assert torch.equal(x[6].view(torch.int32), y[6].view(torch.int32)), f"t={t} average"


@pytest.mark.slow
@pytest.mark.parametrize("U,d", [(1, 5_000_123), (2, 5_000_123), (4, 2_600_077), (8, 1_300_031), (16, 1_300_031), (6, 700_001)])
def test_many_chunks_per_block_with_tiny_layers_between_large_ones(binding, oracle, U, d):
    """Enough chunks that every block of the decoders works through several of them with all its
    teams, and layers of 1, 5 and 130 elements between the large ones (the table changes, and with it
    the whole block synchronises, in the middle of a block's share)."""
    a, b = d // 5, (7 * d) // 10
    off = [0, a, a + 5, a + 135, b, b + 1, d]
    gen = torch.Generator().manual_seed(1000 + U)
    ld = (d + 3) // 4 * 4
    grads = []
    for t in range(2):
        g = torch.zeros((U, ld))
        g[:, :d] = torch.randn((U, d), generator=gen) * (1e-2 if t == 0 else 3e-3)
        g[:, a:a + 135] *= 50.0                              # the tiny layers get their own scale
        grads.append(g.cuda())
    run_case(binding, oracle, d, U, 4, 3, off, grads)


def test_degenerate_values(binding, oracle):
    """All-zero gradient, a constant segment, huge and subnormal values, signed zeros, ties."""
    d = 6000
    g = torch.zeros((2, d))
    g[:, 1000:2000] = 3e-4                               # single-symbol histogram in segment 1
    g[0, 2000:2008] = torch.tensor([1e30, -1e30, 2.0 ** -140, -0.0, 2.0 ** -127, 1e-38, -3e38, 1.0])
    g[1, 2008:4000] = torch.linspace(-1, 1, 1992)
    g[:, 4000:] = torch.arange(2000, dtype=torch.float32) * 2.0 ** -12   # many exact ties
    off = [0, 1000, 2000, 4000, d]
    for E, M in FORMATS:
        run_case(binding, oracle, d, 2, E, M, off, [g.cuda(), (g * -0.5).cuda(), torch.zeros((2, d)).cuda()], gamma=1.0)


def test_nonfinite_inputs(binding, oracle):
    d = 5000
    gen = torch.Generator().manual_seed(3)
    g = torch.randn((2, d), generator=gen) * 1e-3
    g[0, 7] = float("nan"); g[1, 4500] = float("inf"); g[1, 4501] = float("-inf")
    plan, orc, out, res = run_case(binding, oracle, d, 2, 4, 3, [0, 4096, d], [g.cuda(), torch.zeros((2, d)).cuda()])
    flags, nf = plan.status(clear=True)
    assert flags & binding.FLAG_NONFINITE and nf == 3
    assert plan.status() == (0, 0)


@pytest.mark.parametrize("mode", [1, 2])
def test_capacity_overflow_is_flagged_and_stays_inside_the_row(binding, oracle, mode):
    """A payload that does not fit: the flag is raised, offsets and lengths are still complete (they
    are compared with the oracle's inside run_case), and nothing is written past a row's end -- the
    row of the next user and a guard row behind the last one stay as they were."""
    d, U = 20_000, 2
    gen = torch.Generator().manual_seed(4)
    g = (torch.randn((U, d), generator=gen) * 1e-3).cuda()
    plan, orc, out, res = run_case(binding, oracle, d, U, 4, 3, None, [g], cap=1024, mode=mode)
    r, flags = res[0]
    assert r.status == oracle.ECAPACITY and flags & binding.FLAG_CAPACITY
    assert int(out["chunk_off"][0, -1]) > 1024
    # again with a sentinel in the second user's row and a guard row: only user 0's row may change
    plan2 = binding.Plan(d, U, 4, 3, None, bias_mode=mode, cap_words=1024)
    out2 = plan2.alloc_outputs()
    big = torch.full((U + 1, 1024), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    out2["bitstream"] = big[:U]
    plan2.encode(g, torch.zeros_like(g), out2)
    assert plan2.status()[0] & binding.FLAG_CAPACITY
    assert (big[U] == 0x5A5A5A5A).all().item()


def test_corrupt_streams_are_flagged_not_faulting(binding, oracle):
    d, U = 30_000, 3
    gen = torch.Generator().manual_seed(8)
    g = (torch.randn((U, d), generator=gen) * 1e-3).cuda()
    plan, orc, out, res = run_case(binding, oracle, d, U, 4, 3, [0, 10_000, d], [g])
    good = {k: v.clone() for k, v in out.items()}

    def flagged(mut):
        o = {k: v.clone() for k, v in good.items()}
        mut(o)
        plan.status(clear=True)
        plan.decode_aggregate(o)
        return bool(plan.status(clear=True)[0] & binding.FLAG_CORRUPT)

    assert not flagged(lambda o: None)
    assert flagged(lambda o: o["sub_bits"][1, 5].add_(1))
    assert flagged(lambda o: o["chunk_off"][2, 3].add_(2))             # not a multiple of 4
    assert flagged(lambda o: o["chunk_off"][0, 1:].fill_(2 ** 31 - 4))  # far outside the payload
    assert flagged(lambda o: o["hdr"].copy_(binding.hdr_from_numpy(
        binding.hdr_to_numpy(good["hdr"]) + np.array([0, 3, 0]))))      # another code model
    assert flagged(lambda o: o["hdr"].fill_(0x7FFF7F7F))                # indices out of range
    o = {k: v.clone() for k, v in good.items()}                        # random bytes: any outcome but a fault
    o["bitstream"].random_(-2 ** 31, 2 ** 31 - 1)
    plan.decode_aggregate(o)
    torch.cuda.synchronize()
    plan.status(clear=True)
    assert np.array_equal(_bits(plan.decode_aggregate(good).cpu().numpy()),
                          _bits(orc.decode_aggregate(res[0][0].payload, res[0][0].sub_bits,
                                                     res[0][0].chunk_off, res[0][0].hdr)[1]))


@pytest.mark.parametrize("U,E,M", [(3, 4, 3), (12, 3, 2)])
def test_decode_with_fused_model_update(binding, oracle, U, E, M):
    """Algorithm 1 line 14 fused into the decode: w <- fl32(w + fl32(step * avg)), bit for bit, over
    several iterations of a weight vector (both decode kernels: U <= 8 and U > 8)."""
    d, off = 50_001, [0, 4097, 30_000, 50_001]
    gen = torch.Generator().manual_seed(31)
    plan = binding.Plan(d, U, E, M, off)
    orc = oracle.OracleCO3(d, U, E, M, off, cap_words=plan.cap_words)
    out = plan.alloc_outputs()
    m_gpu = torch.zeros((U, plan.ld), device="cuda")
    m_cpu = np.zeros((U, plan.ld), np.float32)
    w_cpu = torch.randn(d, generator=gen).numpy()
    w_gpu = torch.from_numpy(w_cpu.copy()).cuda()
    step = -0.01
    for t in range(3):
        g = torch.zeros((U, plan.ld))
        g[:, :d] = torch.randn((U, d), generator=gen) * 1e-2
        plan.encode(g.cuda(), m_gpu, out)
        r = orc.encode(g.numpy(), m_cpu)
        avg = plan.decode_aggregate_update(out, w_gpu, step).cpu().numpy()
        rc, avg_o = orc.decode_aggregate_update(r.payload, r.sub_bits, r.chunk_off, r.hdr, w_cpu, step)
        assert rc == oracle.OK
        assert np.array_equal(_bits(avg), _bits(avg_o)), f"t={t} average"
        assert np.array_equal(_bits(w_gpu.cpu().numpy()), _bits(w_cpu)), f"t={t} weights"
    assert plan.status()[0] == 0


def test_fit_override_gives_the_oracles_header_from_the_oracles_fit(binding, oracle):
    """Test hook co3_set_fit_override: with the oracle's (beta, alpha) handed in, bias and header come
    out as the oracle's for those numbers, whatever the plan's own moments are; switched off, the
    plan fits its own moments again."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=90_000, n_users=3)
    b = binding
    plan = b.Plan(wl.d, wl.n_users, 4, 3, wl.seg_offsets, gamma=wl.gamma, bias_mode=b.BIAS_CURRENT)
    out = plan.alloc_outputs()
    m = torch.zeros((wl.n_users, plan.ld), dtype=torch.float32, device="cuda")
    g = wl.gradient(0, device="cuda")
    rng = np.random.default_rng(5)
    fit = np.stack([rng.uniform(0.3, 2.0, plan.S), 10.0 ** rng.uniform(-6, 1, plan.S)], axis=1)
    fit[3] = (1.0, 0.0)                                      # a segment declared all-zero
    plan.set_fit_override(fit)
    plan.encode(g, m, out)
    hdr = b.hdr_to_numpy(out["hdr"])
    for l in range(plan.S):
        beta, alpha = float(fit[l, 0]), float(fit[l, 1])
        bias = oracle.bias(beta, alpha, 4, 3)
        assert tuple(hdr[l]) == (bias,) + tuple(oracle.header(beta, alpha, bias)), l
        assert plan.get_fit(l)[:2] == (beta, alpha)
    plan.set_fit_override(None)
    m.zero_()
    plan2 = b.Plan(wl.d, wl.n_users, 4, 3, wl.seg_offsets, gamma=wl.gamma, bias_mode=b.BIAS_CURRENT)
    out2 = plan2.alloc_outputs()
    m2 = torch.zeros_like(m)
    plan.encode(g, m, out)
    plan2.encode(g, m2, out2)
    assert torch.equal(out["hdr"], out2["hdr"]) and torch.equal(out["chunk_off"], out2["chunk_off"])
    for u in range(wl.n_users):                              # (beyond a row's payload lies the first call's)
        n = int(out["chunk_off"][u, -1])
        assert torch.equal(out["bitstream"][u, :n], out2["bitstream"][u, :n])
    with pytest.raises(b.Co3Error):
        plan.set_fit_override(np.full((plan.S, 2), -1.0))


def test_bounded_waits_of_the_encoder_run_out_and_report(binding):
    """Failure detection without a fault: the packing kernel runs with the block of (user 0, chunk 0)
    left out, so nothing publishes that chunk's size; the blocks that need it poll 1000 times, give
    up and return.  The flag is raised, the later chunks are not written, and the same plan encodes
    and decodes normally afterwards."""
    b = binding
    d, U = 3 * 4096, 1
    plan = b.Plan(d, U, 4, 3, None, gamma=0.9)
    out = plan.alloc_outputs()
    m = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(3)
    g = torch.randn((U, plan.ld), generator=gen, device="cuda") * 1e-3
    plan.encode(g, m, out)
    assert plan.status()[0] == 0
    good = {k: v.clone() for k, v in out.items()}
    out["bitstream"].fill_(0x5A5A5A5A)
    plan.debug_encode_stalled(out, spin_limit=1000)
    flags, _ = plan.status(clear=True)
    assert flags & b.FLAG_TIMEOUT
    pay = out["bitstream"].view(-1)
    assert bool((pay == 0x5A5A5A5A).all())                   # chunk 0 was left out, the others gave up
    assert torch.equal(out["sub_bits"][0, 32:], good["sub_bits"][0, 32:])   # lengths do not depend on the waits
    with pytest.raises(b.Co3Error):
        plan.debug_encode_stalled(out, spin_limit=0)
    # the device and the plan are as usable as before
    m.zero_()
    plan2 = b.Plan(d, U, 4, 3, None, gamma=0.9)
    out2 = plan2.alloc_outputs()
    plan2.encode(g, torch.zeros_like(m), out2)
    plan.state_import(0, np.zeros(plan.S, np.int32))
    plan.encode(g, m, out)
    assert plan.status()[0] == 0
    n = int(out["chunk_off"][0, -1])
    assert torch.equal(out["bitstream"][0, :n], good["bitstream"][0, :n])
    assert torch.equal(plan.decode_aggregate(out), plan2.decode_aggregate(out2))


def test_plans_of_one_format_share_their_code_tables(binding):
    """The code tables of all model rows (148 MB for E4M3) exist once per device and format: a second
    plan costs far less device memory than the first, and outlives the first."""
    from paper_2203_09044_b200 import inputs
    b = binding
    wl = inputs.workload(1, d=50_000, n_users=2)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    p1 = b.Plan(wl.d, wl.n_users, 4, 3, wl.seg_offsets, gamma=wl.gamma)
    free1 = torch.cuda.mem_get_info()[0]
    p2 = b.Plan(wl.d, wl.n_users, 4, 3, wl.seg_offsets, gamma=wl.gamma)
    free2 = torch.cuda.mem_get_info()[0]
    assert free1 - free2 < 40 << 20 and (free0 - free1 > 100 << 20 or free0 - free1 < 40 << 20)   # (an earlier test's plan may still hold the tables)
    g = wl.gradient(0, device="cuda")
    outs = []
    for p in (p1, p2):
        out = p.alloc_outputs()
        p.encode(g, torch.zeros((wl.n_users, p.ld), device="cuda"), out)
        outs.append(out)
    assert torch.equal(outs[0]["bitstream"], outs[1]["bitstream"])
    avg1 = p1.decode_aggregate(outs[0]).clone()
    p1.close()
    out = p2.alloc_outputs()
    p2.state_import(0, np.zeros(p2.S, np.int32))
    p2.encode(g, torch.zeros((wl.n_users, p2.ld), device="cuda"), out)
    assert torch.equal(out["bitstream"], outs[0]["bitstream"]) and torch.equal(p2.decode_aggregate(out), avg1)
    assert p2.status()[0] == 0


def test_decoder_depends_only_on_the_stream(binding, oracle):
    """A second plan that never encoded anything (the parameter server) decodes the outputs."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=120_000, n_users=4)
    server = binding.Plan(wl.d, 4, wl.exp_bits, wl.mant_bits, wl.seg_offsets)
    run_case(binding, oracle, wl.d, 4, wl.exp_bits, wl.mant_bits, wl.seg_offsets, _grads(wl, 2),
             decode_plan=server)


def test_run_to_run_determinism_and_state_resume(binding, oracle):
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(2, d=100_003, n_users=4)
    grads = _grads(wl, 4)

    def run(plan, m, ts):
        outs = []
        for t in ts:
            out = plan.alloc_outputs()
            plan.encode(grads[t], m, out)
            plan.decode_aggregate(out)
            outs.append({k: v.clone() for k, v in out.items()})
        return outs

    mk = lambda: binding.Plan(wl.d, 4, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma)
    z = lambda p: torch.zeros((4, p.ld), device="cuda")
    p1, p2 = mk(), mk()
    m1, m2 = z(p1), z(p2)
    a = run(p1, m1, range(4))
    b2 = run(p2, m2, range(2))
    it, nb = p2.state_export()
    assert it == 2
    p3 = mk()
    p3.state_import(it, nb)                              # resume on a fresh plan with the saved memory
    b2 += run(p3, m2, range(2, 4))
    for x, y in zip(a, b2):
        for k in x:
            assert torch.equal(x[k], y[k]), k
    assert torch.equal(m1, m2)


def test_host_iteration_entry_point(binding, oracle):
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(0, d=50_000, n_users=2)
    plan = binding.Plan(wl.d, 2, 4, 3)
    orc = oracle.OracleCO3(wl.d, 2, 4, 3, cap_words=plan.cap_words)
    out = plan.alloc_outputs()
    m = torch.zeros((2, plan.ld), device="cuda")
    m_cpu = np.zeros((2, plan.ld), np.float32)
    d_grad = torch.empty((2, plan.ld), device="cuda")
    h_avg = torch.empty(wl.d).pin_memory()
    for t in range(2):
        h_grad = wl.gradient(t).pin_memory()
        plan.iteration_host(h_grad, d_grad, m, out, h_avg)
        torch.cuda.synchronize()
        r = orc.encode(h_grad.numpy().copy(), m_cpu)
        rc, avg_o, _ = orc.decode_aggregate(r.payload, r.sub_bits, r.chunk_off, r.hdr)
        assert np.array_equal(_bits(h_avg.numpy()), _bits(avg_o))


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("tile", [1, 2, 4])
def test_iteration_in_tiles_of_users(binding, oracle, mode, tile):
    """The gradient supplied in tiles of users through ONE reused tile buffer (co3_tiled_*): every
    output of every iteration is bit for bit what the oracle gets from the whole gradient."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=90_000, n_users=5)
    plan = binding.Plan(wl.d, 5, 4, 3, wl.seg_offsets, bias_mode=mode)
    orc = oracle.OracleCO3(wl.d, 5, 4, 3, wl.seg_offsets, mode=mode, cap_words=plan.cap_words)
    out = plan.alloc_outputs()
    m_gpu = torch.zeros((5, plan.ld), device="cuda")
    m_cpu = np.zeros((5, plan.ld), np.float32)
    buf = torch.empty((tile, plan.ld), device="cuda")
    for t in range(4):
        # (the scale moves, and a few elements of the later users lie far beyond the previous iteration's range:
        # with the bias from the current moments the tiles are converted under the previous bias, every layer is
        # converted again in co3_tiled_finish, and those elements come from the side list)
        g = wl.gradient(t) * (1.0, 8.0, 0.25, 1.0)[t]
        if t % 2 == 1:
            g[3, 5000:5010] = 1e12
            g[4, 70_000] = -1e12

        def make_tile(u0, n):
            buf[:n].copy_(g[u0:u0 + n])
            return buf

        plan.encode_tiled(tile, make_tile, m_gpu, out)
        r = orc.encode(g.numpy(), m_cpu)
        compare_iteration(binding, plan, out, r, m_gpu, m_cpu, tag=f"tile={tile} t={t}")
        avg = plan.decode_aggregate(out).cpu().numpy()
        rc, avg_o, _ = orc.decode_aggregate(r.payload, r.sub_bits, r.chunk_off, r.hdr)
        assert rc == oracle.OK and np.array_equal(_bits(avg), _bits(avg_o))
    assert plan.status()[0] == 0
    # misuse is refused: a convert tile before the statistics tiles, a user twice, a finish too early
    fresh = binding.Plan(wl.d, 5, 4, 3, wl.seg_offsets, bias_mode=mode)
    L = binding.lib()
    import ctypes as C
    need = C.c_int32()
    assert L.co3_tiled_begin(fresh.handle, C.byref(need)) == 0 and need.value == 1
    p_buf, p_m = C.c_void_p(buf.data_ptr()), C.c_void_p(m_gpu.data_ptr())
    assert L.co3_tiled_convert(fresh.handle, p_buf, p_m, 0, 1, None) == binding.EINVAL
    assert L.co3_tiled_statistics(fresh.handle, p_buf, p_m, 4, 2, None) == binding.EINVAL   # beyond the last user
    o = fresh.alloc_outputs()
    ptrs = [C.c_void_p(o[k].data_ptr()) for k in ("bitstream", "sub_bits", "chunk_off", "user_bits", "hdr")]
    assert L.co3_tiled_finish(fresh.handle, *ptrs, None) == binding.EINVAL


@pytest.mark.parametrize("mode", [1, 0])
def test_steady_state_iteration_replays_from_a_cuda_graph(binding, oracle, mode):
    """After the first iteration (which has the extra statistics pass) an iteration is a fixed
    sequence of memsets and kernels on one stream with no host decision in it, so it can be captured
    once in a CUDA graph and replayed: the replays, fed through the captured input buffer, must be
    the oracle's iterations bit for bit (state carried in device memory: residual, bias, tickets).
    With the bias from the current moments (mode 0) the layers whose bias changed are found and
    converted again on the device; the gradients' scale moves between the replays so that some are."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=120_000, n_users=3)
    plan = binding.Plan(wl.d, 3, 4, 3, wl.seg_offsets, bias_mode=mode)
    orc = oracle.OracleCO3(wl.d, 3, 4, 3, wl.seg_offsets, cap_words=plan.cap_words, mode=mode)
    scale = (1.0, 1.0, 6.0, 0.5)
    out = plan.alloc_outputs()
    m = torch.zeros((3, plan.ld), device="cuda")
    m_cpu = np.zeros((3, plan.ld), np.float32)
    g_static = wl.gradient(0).cuda()                    # (drawn on the CPU: the same numbers as the oracle's)
    plan.encode(g_static, m, out)                       # t = 0, eager
    plan.decode_aggregate(out)
    orc.encode(wl.gradient(0).numpy(), m_cpu)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):                       # t = 1 is captured (and not run)
        plan.encode(g_static, m, out)
        plan.decode_aggregate(out)
    for t in range(1, 4):
        g_static.copy_(wl.gradient(t) * scale[t])
        graph.replay()
        torch.cuda.synchronize()
        r = orc.encode((wl.gradient(t) * scale[t]).numpy(), m_cpu)
        rc, avg_o, _ = orc.decode_aggregate(r.payload, r.sub_bits, r.chunk_off, r.hdr)
        assert rc == oracle.OK
        assert np.array_equal(b_hdr(binding, out), r.hdr), f"t={t} header"
        n = int(out["chunk_off"][0, -1])
        assert np.array_equal(out["bitstream"].cpu().numpy().view(np.uint32)[0, :n], r.payload[0, :n]), f"t={t}"
        assert np.array_equal(_bits(out["avg"].cpu().numpy()), _bits(avg_o)), f"t={t} average"
        assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_cpu)), f"t={t} memory"
    assert plan.status()[0] == 0


def b_hdr(binding, out):
    return binding.hdr_to_numpy(out["hdr"])


def test_host_iterations_back_to_back_overlap_their_copies(binding, oracle):
    """Four co3_iteration_host calls enqueued without any synchronisation in between (the copies of
    one call overlap the work of the previous one on the plan's own streams): every average and
    the final memory must still be the oracle's."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, d=1_500_000, n_users=4)
    plan = binding.Plan(wl.d, 4, 4, 3, wl.seg_offsets)
    orc = oracle.OracleCO3(wl.d, 4, 4, 3, wl.seg_offsets, cap_words=plan.cap_words)
    out = plan.alloc_outputs()
    m = torch.zeros((4, plan.ld), device="cuda")
    m_cpu = np.zeros((4, plan.ld), np.float32)
    d_grad = torch.empty((4, plan.ld), device="cuda")
    h_grads = [wl.gradient(t).pin_memory() for t in range(4)]
    h_avgs = [torch.empty(wl.d).pin_memory() for _ in range(4)]
    for t in range(4):
        plan.iteration_host(h_grads[t], d_grad, m, out, h_avgs[t])
    torch.cuda.synchronize()
    for t in range(4):
        r = orc.encode(h_grads[t].numpy().copy(), m_cpu)
        rc, avg_o, _ = orc.decode_aggregate(r.payload, r.sub_bits, r.chunk_off, r.hdr)
        assert rc == oracle.OK and np.array_equal(_bits(h_avgs[t].numpy()), _bits(avg_o)), f"t={t}"
    assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_cpu))
    assert plan.status()[0] == 0


# ---- full sizes, in the launch configuration the benchmark times ---------------------------
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("world", [2, 3])
def test_slices_of_d_with_pooled_moments_equal_the_whole(binding, oracle, mode, world):
    """The gradient cut into `world` slices of d, one plan per slice (as one GPU per slice would hold
    them), run phase by phase on this GPU with the slices' moment tables added between the phases
    (what the all-reduce does): payload, side information, headers, memory and average of the
    slices, put end to end, are those of the oracle on the whole gradient."""
    from paper_2203_09044_b200 import inputs, sharded
    wl = inputs.workload(1, d=150_000, n_users=3)
    U, d, off = wl.n_users, wl.d, wl.seg_offsets
    orc = oracle.OracleCO3(d, U, 4, 3, off, gamma=wl.gamma, mode=mode)
    ranks = [sharded.ShardedPlan(d, U, 4, 3, off, r, world, gamma=wl.gamma, bias_mode=mode) for r in range(world)]
    assert sum(len(sp.layout.seg_ids) for sp in ranks) > len(off) - 1      # some layer spans a cut
    outs = [sp.plan.alloc_outputs() for sp in ranks]
    m_gpu = [torch.zeros((U, sp.plan.ld), dtype=torch.float32, device="cuda") for sp in ranks]
    m_cpu = np.zeros((U, wl.ld), np.float32)
    for t in range(3):
        g = wl.gradient(t, device="cuda") * (1.0, 6.0, 0.5)[t]      # (so that the biases move)
        gs = []
        for sp in ranks:
            x = torch.zeros((U, sp.plan.ld), dtype=torch.float32, device="cuda")
            x[:, :sp.plan.d] = g[:, sp.layout.lo:sp.layout.hi]
            gs.append(x)
        need = [sp.begin() for sp in ranks]
        assert need == [t == 0] * world              # (the current-moments bias converts under the previous bias and repairs)
        pooled = None
        if need[0]:
            pooled = sum(sp.statistics(gs[r], m_gpu[r]) for r, sp in enumerate(ranks))
        pooled = sum(sp.convert(gs[r], m_gpu[r], pooled) for r, sp in enumerate(ranks))
        for r, sp in enumerate(ranks):
            sp.finish(pooled, outs[r])
        ro = orc.encode(g.cpu().numpy(), m_cpu)
        assert np.array_equal(pooled.cpu().numpy()[:, 0], ro.moments[:, 0]), f"t={t} pooled counts"
        np.testing.assert_allclose(pooled.cpu().numpy()[:, 1:], ro.moments[:, 1:], rtol=1e-12)
        m_all = np.concatenate([m.cpu().numpy()[:, :sp.plan.d] for m, sp in zip(m_gpu, ranks)], axis=1)
        assert np.array_equal(_bits(m_all), _bits(m_cpu[:, :d])), f"t={t} residual"
        for r, sp in enumerate(ranks):
            hdr = binding.hdr_to_numpy(outs[r]["hdr"])
            assert np.array_equal(hdr, ro.hdr[sp.layout.seg_ids]), f"t={t} header of slice {r}"
        cos = [o["chunk_off"].cpu().numpy().view(np.uint32) for o in outs]
        pays = [o["bitstream"].cpu().numpy().view(np.uint32) for o in outs]
        for u in range(U):
            words = np.concatenate([pays[r][u, :int(cos[r][u, -1])] for r in range(world)])
            assert int(ro.chunk_off[u, -1]) == len(words)
            assert np.array_equal(words, ro.payload[u, :len(words)]), f"t={t} payload of user {u}"
            base, offs = 0, []
            for r in range(world):
                offs.append(cos[r][u, :-1].astype(np.int64) + base)
                base += int(cos[r][u, -1])
            assert np.array_equal(np.concatenate(offs), ro.chunk_off[u, :-1]), f"t={t} chunk offsets"
        sb = np.concatenate([o["sub_bits"].cpu().numpy().view(np.uint16)[:, :sp.plan.n_sub]
                             for o, sp in zip(outs, ranks)], axis=1)
        assert np.array_equal(sb, ro.sub_bits[:, :sb.shape[1]]), f"t={t} sub_bits"
        ub = sum(o["user_bits"].cpu().numpy().view(np.uint64) for o in outs)
        assert np.array_equal(ub, ro.user_bits), f"t={t} user_bits"
        avg = np.concatenate([sp.decode_aggregate(outs[r]).cpu().numpy()[:sp.plan.d] for r, sp in enumerate(ranks)])
        rc, avg_o, _ = orc.decode_aggregate(ro.payload, ro.sub_bits, ro.chunk_off, ro.hdr)
        assert rc == oracle.OK and np.array_equal(_bits(avg), _bits(avg_o)), f"t={t} averaged gradient"
        for sp in ranks:
            assert sp.plan.status()[0] == 0


def test_moments_calls_are_refused_outside_their_places(binding):
    plan = binding.Plan(10_000, 2, 4, 3)
    mom = torch.zeros((1, 3), dtype=torch.float64, device="cuda")
    with pytest.raises(binding.Co3Error):
        plan.moments_export(mom)                                  # no tiled iteration open
    assert plan.tiled_begin()
    with pytest.raises(binding.Co3Error):
        plan.moments_import(mom)                                  # before any statistics tile
    g = torch.randn((2, plan.ld), device="cuda") * 1e-3
    m = torch.zeros_like(g)
    plan.tiled_statistics(g, m, 0, 1)
    plan.tiled_statistics(g, m, 1, 1)
    own = plan.moments_export().cpu().numpy()
    assert own[0, 0] == 2 * 10_000 and own[0, 1] > 0 and own[0, 2] > 0
    plan.tiled_convert(g, m, 0, 1)
    with pytest.raises(binding.Co3Error):
        plan.moments_export(mom)                                  # a user is still to be converted
    plan.tiled_convert(g, m, 1, 1)
    out = plan.alloc_outputs()
    plan.tiled_finish(out)                                        # without an import: the plan's own sums
    assert plan.status()[0] == 0


def test_moments_export_of_a_very_long_segment(binding):
    """A segment with more than 2^15 (user, chunk) pairs is summed in slices first; the exported sums
    are those of a plain fp64 sum over the inputs, and exactly the ones the fit then reports."""
    U, d = 64, 2_200_000
    plan = binding.Plan(d, U, 3, 2)
    gen = torch.Generator(device="cuda").manual_seed(5)
    g = torch.randn((U, plan.ld), generator=gen, device="cuda") * 2e-3
    g[:, d:] = 0
    m = torch.zeros_like(g)
    assert plan.tiled_begin()
    plan.tiled_statistics(g, m, 0, U)
    mom = plan.moments_export().cpu().numpy()
    a = g[:, :d].double()
    assert mom[0, 0] == U * d
    np.testing.assert_allclose(mom[0, 1:], [float(a.abs().sum()), float((a * a).sum())], rtol=1e-12)
    plan.tiled_convert(g, m, 0, U)
    mom2 = plan.moments_export().cpu().numpy()
    out = plan.alloc_outputs()
    plan.tiled_finish(out)
    beta, alpha, N, S1, S2 = plan.get_fit(0)
    assert (N, S1, S2) == tuple(mom2[0]) and plan.status()[0] == 0
    np.testing.assert_allclose(mom2[0], mom[0], rtol=1e-12)          # same a = g + gamma * 0 in both passes


@pytest.mark.slow
def test_config0_full(binding, oracle):
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(0)
    run_case(binding, oracle, wl.d, wl.n_users, 4, 3, wl.seg_offsets, _grads(wl, wl.iters), gamma=wl.gamma)


@pytest.mark.slow
def test_config1_full_two_iterations(binding, oracle):
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1).align_rows()           # rows on 16 KiB boundaries, as the benchmark lays them out
    run_case(binding, oracle, wl.d, wl.n_users, 4, 3, wl.seg_offsets, _grads(wl, 2), gamma=wl.gamma)


@pytest.mark.slow
@pytest.mark.parametrize("mode,rule", [(0, 0), (2, 0), (3, 0), (1, 1)])
def test_config1_full_other_modes_two_iterations(binding, oracle, mode, rule):
    """Configuration 1 at full size with the bias from the current moments (three iterations: the second
    and third convert under the previous bias and repair the layers whose bias changed), in the fully
    lagged-code mode, the empirical-histogram mode and with the L2-optimal bias rule (two iterations
    each: the second one runs on carried state)."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1).align_rows()
    run_case(binding, oracle, wl.d, wl.n_users, 4, 3, wl.seg_offsets, _grads(wl, 3 if mode == 0 else 2), gamma=wl.gamma,
             mode=mode, rule=rule)


@pytest.mark.slow
def test_config2_full_two_iterations(binding, oracle):
    """16 users x d = 14,728,266 in 16 segments with odd offsets, E3M2 (the U > 8 decode path).  The
    second iteration runs on the carried memory with the bias of the first one's fit (Algorithm 1
    lines 8 and 10 feed iteration t + 1)."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(2)
    run_case(binding, oracle, wl.d, wl.n_users, 3, 2, wl.seg_offsets, _grads(wl, 2), gamma=wl.gamma)


@pytest.mark.slow
def test_config3_full_two_iterations(binding, oracle):
    """4 users x d = 124,439,808 heavy-tailed with outliers, E4M3: the shape estimate clamps at 0.3.
    Two iterations, so that the sliced moment reduction of a very long segment also runs on carried
    state (no statistics pass, non-zero memory, lagged bias)."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(3)
    plan, orc, out, res = run_case(binding, oracle, wl.d, wl.n_users, 4, 3, wl.seg_offsets, _grads(wl, 2),
                                   gamma=wl.gamma)
    assert res[0][0].fit[0, 0] == 0.3 and res[1][0].fit[0, 0] == 0.3


# ---- the size / users / shape / format sweep (a subset the oracle can follow) ----------------
@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("beta", [0.5, 1.0, 2.0])
@pytest.mark.parametrize("U", [1, 8, 64])
def test_sweep_d_2p16(binding, oracle, U, beta, E, M):
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 16, U, beta, E, M)
    run_case(binding, oracle, wl.d, U, E, M, wl.seg_offsets, _grads(wl, 2), gamma=wl.gamma)


@pytest.mark.slow
@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("beta", [0.5, 2.0])
def test_sweep_d_2p20_8_users(binding, oracle, beta, E, M):
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 20, 8, beta, E, M)
    run_case(binding, oracle, wl.d, 8, E, M, wl.seg_offsets, _grads(wl, 1), gamma=wl.gamma)


@pytest.mark.slow
@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("U", [1, 8, 64])
def test_sweep_d_2p20_laplace_shape(binding, oracle, U, E, M):
    """d = 2^20 with 1, 8 and 64 users at beta = 1.0, two iterations (the second on carried state)."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 20, U, 1.0, E, M)
    run_case(binding, oracle, wl.d, U, E, M, wl.seg_offsets, _grads(wl, 2), gamma=wl.gamma)


@pytest.mark.slow
@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("beta", [0.5, 1.0, 2.0])
def test_sweep_d_2p24_8_users(binding, oracle, beta, E, M):
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 24, 8, beta, E, M)
    run_case(binding, oracle, wl.d, 8, E, M, wl.seg_offsets, _grads(wl, 1), gamma=wl.gamma)


@pytest.mark.slow
@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("beta", [0.5, 1.0, 2.0])
def test_sweep_d_2p24_single_user_all_shapes(binding, oracle, beta, E, M):
    """One user: the decoder of its own (24 independent warps per block), 4096 chunks."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 24, 1, beta, E, M)
    run_case(binding, oracle, wl.d, 1, E, M, wl.seg_offsets, _grads(wl, 1), gamma=wl.gamma)


@pytest.mark.slow
@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("beta", [0.5, 2.0])
@pytest.mark.parametrize("U", [1, 64])
def test_sweep_d_2p20_other_shapes(binding, oracle, U, beta, E, M):
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 20, U, beta, E, M)
    run_case(binding, oracle, wl.d, U, E, M, wl.seg_offsets, _grads(wl, 1), gamma=wl.gamma)


@pytest.mark.slow
def test_sweep_d_2p24_64_users_fp4(binding, oracle):
    """The one U = 64 cell above 2^16 that the oracle can follow in about two minutes: 4096 chunks of 64
    streams each, so every block of the many-user decoder walks dozens of chunks."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.sweep_cell(1 << 24, 64, 1.0, 1, 2)
    run_case(binding, oracle, wl.d, 64, 1, 2, wl.seg_offsets, _grads(wl, 1), gamma=wl.gamma)


@pytest.mark.slow
def test_sweep_d_2p24_and_2p28_single_user(binding, oracle):
    from paper_2203_09044_b200 import inputs
    for d, E, M in ((1 << 24, 3, 2), (1 << 28, 1, 2)):
        wl = inputs.sweep_cell(d, 1, 1.0, E, M)
        run_case(binding, oracle, wl.d, 1, E, M, wl.seg_offsets, _grads(wl, 1), gamma=wl.gamma)
