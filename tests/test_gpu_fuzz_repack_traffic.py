"""Seeded random descriptors through ccl_repack and ccl_traffic against the oracle, bit for bit: element sizes, strip
counts (equal and unequal strips), row / column splits, packed, aligned and page-interleaved layouts, both directions,
both repack kernels; tile sizes, page sizes, placements, tile-to-chiplet assignments.  Descriptors either side rejects are
rejected by both."""
import random

import numpy as np
import pytest

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from helpers import mat_pair, traffic_pair
from test_gpu_repack_traffic import run_repack, run_traffic

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [1, 2])
def test_random_repack_descriptors(seed):
    rng = random.Random(seed)
    done = rejected = 0
    while done < 150:
        e = rng.choice([1, 2, 2, 4])
        rows, cols = rng.choice([1, 2, 7, 33, 64, 130, 257, 512]), rng.choice([8, 16, 50, 96, 200, 384, 520, 1000, 1536])
        P, part, layout = rng.choice([1, 2, 3, 4, 5, 8]), rng.choice([1, 2, 2]), rng.choice([1, 1, 2])
        align = rng.choice([16, 64, 256, 1024, 4096]) if layout == 2 else rng.choice([0, 0, 16, 128, 1024, 4096])
        case = dict(rows=rows, cols=cols, e=e, P=P, part=part, layout=layout, align=align)
        try:
            mo, ml = mat_pair(**case)
            n_o = orc.buffer_bytes(mo)
        except Exception:
            n_o = None
        try:
            n_l = ccl.ccl_buffer_bytes(mat_pair(**case)[1])
        except ccl.CclError:
            n_l = None
        assert (n_o is None) == (n_l is None), case      # both sides agree on what is a legal descriptor
        if n_o is None:
            rejected += 1
            continue
        assert n_o == n_l, case
        run_repack(case, path=rng.choice(["vec", "tma", None]), seed=done)
        done += 1
    assert rejected < 10 * done


@pytest.mark.parametrize("seed", [1, 2])
def test_random_traffic_descriptors(seed):
    rng = random.Random(seed)
    done = 0
    while done < 60:
        P = rng.choice([1, 2, 3, 4, 6, 8])
        assign = rng.choice([0, 0, 1, 3])
        part_m = rng.choice([d for d in (1, 2, 3, 4) if P % d == 0]) if assign == 3 else 0
        shape = dict(M=rng.choice([1, 16, 97, 130, 256]), N=8 * rng.randint(4, 64), K=8 * rng.randint(2, 24), P=P,
                     S=rng.choice([16, 48, 128, 256, 4096, 1 << 21]), BM=rng.choice([16, 32, 128]), BN=rng.choice([32, 64, 128]),
                     a_trans=rng.choice([0, 1]), b_trans=rng.choice([0, 1]), assign=assign, part_m=part_m, strip_tiling=rng.choice([0, 1]))
        lay = rng.choice([("row", "row", "row"), ("row", "ccl", "ccl"), ("ccl", "ccl", "ccl"), ("row", "ileave", "ileave")])
        place = tuple(rng.choice([0, 1, 2]) for _ in range(3))
        align = rng.choice([64, 1024]) if "ileave" in lay else rng.choice([0, 1024])
        try:
            do, dl = traffic_pair(lay=lay, place=place, align=align, **shape)
            orc.traffic_sizes(do)
        except Exception:
            continue                                     # (e.g. a partition that would leave a strip empty)
        run_traffic(do, dl, "elem")
        done += 1
