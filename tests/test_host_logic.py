"""CPU-only checks of the CUDA library's host side: it loads, exports what include/co3.h
declares, rejects bad configurations before touching CUDA, and its two host-computed tables (the
static partition and the GenNorm model-weight table) are identical to the oracle's own."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2203_09044_b200 import build, binding as b
    build.build()
    b.lib()
    return b


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "co3.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(co3_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    L = binding.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert L.co3_strerror(0) == b"ok" and b"capacity" not in L.co3_strerror(-1)


def test_bad_configurations_are_rejected_on_the_host(binding):
    L = binding.lib()

    def create(**kw):
        base = dict(d=1000, ld=1000, n_users=2, E=4, M=3, gamma=0.9, mode=1, cap=4000, off=None)
        base.update(kw)
        off = None if base["off"] is None else np.asarray(base["off"], np.int64)
        cfg = binding.Config(base["d"], base["ld"], base["n_users"], binding.Format(base["E"], base["M"]),
                             0 if off is None else len(off) - 1,
                             None if off is None else off.ctypes.data_as(C.POINTER(C.c_int64)),
                             base["gamma"], base["mode"], base["cap"], base.get("rule", 0), 0)
        h = C.c_void_p()
        rc = L.co3_plan_create(C.byref(h), C.byref(cfg))
        if rc == 0:
            L.co3_plan_destroy(h)
        return rc

    assert create(d=0) == binding.EINVAL
    assert create(ld=998) == binding.EINVAL and create(ld=1002) == binding.EINVAL
    assert create(E=5) == binding.EINVAL and create(M=0) == binding.EINVAL and create(E=4, M=4) == binding.EINVAL
    assert create(n_users=0) == binding.EINVAL
    assert create(n_users=69) == binding.EINVAL          # 69 * 245760 >= 2^24: sums not exact
    assert create(cap=4001) == binding.EINVAL and create(cap=0) == binding.EINVAL
    assert create(gamma=1.5) == binding.EINVAL and create(mode=7) == binding.EINVAL
    assert create(rule=2) == binding.EINVAL
    assert create(off=[0, 600, 500, 1000]) == binding.EINVAL
    assert create(off=[0, 500, 900]) == binding.EINVAL
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if not has_gpu:                                      # a valid plan needs a device: clean error
        assert create() in (binding.ENOMEM, binding.ECUDA)


@pytest.mark.parametrize("E,M", [(1, 2), (3, 2), (4, 3)])
def test_model_weight_table_identical_to_oracle(binding, oracle, E, M):
    """The code tables of both sides are built from these integers: they must agree exactly for
    every header index pair."""
    for ib in range(-14, 9):
        for ir in range(-96, 32):
            a = binding.model_weights(E, M, ib, ir)
            b = oracle.model_weights(E, M, ib, ir)
            assert np.array_equal(a, b), (ib, ir, np.nonzero(a != b))
    with pytest.raises(binding.Co3Error):
        binding.model_weights(E, M, 9, 0)


def test_model_checksum_is_the_digest_of_the_weight_table(binding):
    """What two hosts compare before the first iteration: FNV-1a over all 23 x 128 rows of non-negative
    magnitudes, recomputed here from co3_model_weights."""
    for E, M in [(1, 2), (3, 2), (4, 3)]:
        J = 1 << (E + M)
        h = 0xcbf29ce484222325
        for ib in range(-14, 9):
            for ir in range(-96, 32):
                for byte in binding.model_weights(E, M, ib, ir)[:J].astype("<u4").tobytes():
                    h = ((h ^ byte) * 0x100000001b3) & 0xFFFFFFFFFFFFFFFF
        assert binding.model_checksum(E, M) == h != 0
    assert binding.model_checksum(5, 3) == 0
    assert len({binding.model_checksum(E, M) for E, M in [(1, 2), (3, 2), (4, 3)]}) == 3


def _block_cost(w, seg, a, z, teams):
    """Time of the items a .. z-1 in one block, as co3_balanced_split defines it."""
    total, i = 0.0, a
    while i < z:
        j = i
        while j < z and seg[j] == seg[i]:
            j += 1
        team_max = max(float(np.sum(w[i + t:j:teams])) for t in range(teams))
        total += 0.5 * team_max + 0.5 * float(np.sum(w[i:j])) / teams + 0.04
        i = j
    return total


def test_balanced_split_of_the_decoders_work(binding):
    """The cuts cover the items in order, use at most max_blocks blocks, and their largest block cost
    is the least any contiguous split reaches (brute force on small cases); on the ResNet-18 layer mix
    it beats equal item counts per block."""
    import itertools
    from paper_2203_09044_b200 import inputs
    rng = np.random.default_rng(3)
    for n, blocks, teams in ((9, 3, 2), (11, 4, 4), (7, 7, 1), (10, 2, 3), (5, 8, 4)):
        w = rng.choice([0.04 + 1.0, 0.04 + 0.5, 0.04 + 0.1], n)
        seg = np.sort(rng.integers(0, 3, n)).astype(np.int32)
        part, nb = binding.balanced_split(w, seg, teams, blocks)
        assert part[0] == 0 and part[nb] == n and np.all(np.diff(part[:nb + 1]) > 0) and np.all(part[nb:] == n)
        got = max(_block_cost(w, seg, part[b], part[b + 1], teams) for b in range(nb))
        best = min(max(_block_cost(w, seg, a, z, teams) for a, z in zip((0,) + cuts, cuts + (n,)))
                   for k in range(0, min(blocks, n)) for cuts in itertools.combinations(range(1, n), k))
        assert got <= best + 1e-9, (n, blocks, teams, got, best)
    wl = inputs.workload(1)
    seg, st, en, _, _ = binding.partition(wl.d, wl.seg_offsets)
    w = 0.04 + np.minimum(en - st, 128) / 128.0
    part, nb = binding.balanced_split(w, seg, 4, 148)
    balanced = max(_block_cost(w, seg, part[b], part[b + 1], 4) for b in range(nb))
    per = -(-len(seg) // 148)
    equal = max(_block_cost(w, seg, a, min(a + per, len(seg)), 4) for a in range(0, len(seg), per))
    assert nb == 148 and balanced < 0.9 * equal, (nb, balanced, equal)
    with pytest.raises(binding.Co3Error):
        binding.balanced_split(w, seg, 33, 148)


def test_partition_identical_to_oracle(binding, oracle):
    from paper_2203_09044_b200 import inputs
    cases = [(10000, [0, 10000]), (9000, [0, 5, 5, 4101, 8192, 9000]), (130, [0, 1, 130]),
             (1, [0, 1]), (4096, [0, 4096])]
    w1, w2 = inputs.workload(1), inputs.workload(2)
    cases += [(w1.d, w1.seg_offsets), (w2.d, w2.seg_offsets)]
    for d, off in cases:
        seg, st, en, sb, ns = binding.partition(d, off)
        p = oracle.Partition(d, off)
        assert ns == p.n_sub and len(seg) == p.n_chunks
        n = p.n_chunks
        assert np.array_equal(seg, p.chunk_seg[:n]) and np.array_equal(st, p.chunk_start[:n])
        assert np.array_equal(en, p.chunk_end[:n]) and np.array_equal(sb, p.sub_base[:n])


def test_sweep_report_helpers_need_no_gpu():
    """The throughput report module: which workloads it would skip for lack of device memory, and
    one formatted table row (no GPU is touched by these helpers)."""
    from paper_2203_09044_b200 import inputs, sweep
    big = inputs.sweep_cell(1 << 28, 64, 1.0, 4, 3)
    small = inputs.sweep_cell(1 << 16, 8, 1.0, 1, 2)
    assert sweep.device_bytes_needed(big, 1) > 150e9 > 60e9 > sweep.device_bytes_needed(small, 2)
    r = dict(name="x", d=1 << 20, U=8, S=1, fmt="E4M3", beta=1.0, ms=0.5, first_ms=1.0, gbs=67.1, convert_ms=0.02,
             encode_ms=0.03, fit_ms=0.01, decode_ms=0.03, code_bits=6.8, container_bits=6.95, flags=0, l2_resident=True)
    cells = [c.strip() for c in sweep.row(r, 6550.7).split("|")]
    assert cells[1] == "x" and cells[4] == "E4M3" and "launch-bound" in cells[-2]
    assert float(cells[-5]) == 0.0                      # no realised error given: column printed as 0
    # Huffman cost from counts: sum of internal node weights; dyadic counts cost exactly the entropy
    assert sweep.huffman_cost([8, 4, 2, 1, 1]) == 8 * 1 + 4 * 2 + 2 * 3 + 1 * 4 + 1 * 4
    assert sweep.huffman_cost([5, 0, 0]) == 5.0 and sweep.huffman_cost([3, 3, 3, 3]) == 24.0
    conv_gbs = 13.0 * 8 * (1 << 20) / 0.02e-3 / 1e9
    assert abs(float(cells[9]) - round(conv_gbs)) <= 1


@pytest.mark.parametrize("E,M", [(1, 2), (3, 2), (4, 3)])
def test_optimal_bias_table_is_identical_in_library_and_oracle(binding, oracle, E, M):
    """The 23 x 8 table behind the L2-optimal bias rule, and the objective it is the argmin of, from
    the library's own incomplete-gamma code and from the oracle's: same choices everywhere, same
    distortion to 1e-9."""
    assert np.array_equal(binding.bias_opt_table(E, M), oracle.bias_opt_table(E, M))
    for ib in (-14, -5, 0, 3, 8):
        for ir in (-96, -40, -17, -3, 0, 9, 31):
            a, b = binding.grid_distortion(E, M, ib, ir), oracle.distortion(E, M, ib, ir)
            assert a > 0 and abs(a - b) <= 1e-9 * b
    assert binding.grid_distortion(E, M, 9, 0) < 0 and binding.grid_distortion(E, M, 0, 32) < 0


def test_bench_reads_the_convert_traffic_from_the_profile_record():
    """roofline.traffic of the bench line comes from the figures kept beside the ncu summary, scaled
    by the number of users; algorithmic bytes of the convert pass are 13 per user-element."""
    import json
    import sys
    sys.path.insert(0, ROOT)
    import bench
    rec = json.load(open(os.path.join(ROOT, "profiles", "dram_traffic_config1_8users.json")))
    assert bench.convert_dram_traffic(8) == rec["convert_dram_bytes_per_launch"]
    assert bench.convert_dram_traffic(2) == rec["convert_dram_bytes_per_launch"] / 4
    algorithmic = bench.CONVERT_BYTES_PER_ELEMENT * 8 * 11_173_962
    assert 0.9 * algorithmic < rec["convert_dram_bytes_per_launch"] < 1.05 * algorithmic
