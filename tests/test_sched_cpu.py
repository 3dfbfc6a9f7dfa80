"""Host-side check of the tile scheduler's work list (psa_sched.h compiled with g++): with and without the tail of
single row tiles, every (batch*head, row tile) appears in exactly one item, items own one or two consecutive tiles of
one head, and the split rule only fires where it can help."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = r"""
#include <cstdio>
#include <cstdlib>
#include <vector>
#include "paper_2012_01114_b200/csrc/psa_sched.h"
using namespace psa;
int main(int argc, char** argv) {
    const int scheme = atoi(argv[1]), nbh = atoi(argv[2]), n = atoi(argv[3]), d = atoi(argv[4]), sms = atoi(argv[5]);
    const int T = row_tiles(n), P = ctas_per_head(n);
    const long long pairs = (long long)nbh * P;
    const long long split = split_point(scheme, pairs, n, sms);
    const long long nitems = pairs + (pairs - split);
    const int group = lpt_group(scheme, nbh, n, d);
    std::vector<int> seen((size_t)nbh * T, 0);
    long long singles = 0;
    const SchedParams sp = sched_params(n, scheme == PSA_MASKED, nbh, group, split == pairs ? 0x7fffffff : (int)split);
    for (long long i = 0; i < nitems; ++i) {
        const CtaWork w = split == pairs ? cta_work((int)i, n, scheme == PSA_MASKED, nbh, group)
                                         : cta_work_split((int)i, n, scheme == PSA_MASKED, nbh, group, (int)split);
        const CtaWork f = item_work_fast(sp, (int)i);      // the division-free decoding the kernel uses
        if (f.bh != w.bh || f.tile0 != w.tile0 || f.ntiles != w.ntiles) return 5;
        if (w.bh < 0 || w.bh >= nbh || w.ntiles < 1 || w.ntiles > 2 || w.tile0 < 0 || w.tile0 + w.ntiles > T) return 2;
        if (i >= split && w.ntiles != 1) return 3;
        if (i >= split) ++singles;
        for (int t = 0; t < w.ntiles; ++t) ++seen[(size_t)w.bh * T + w.tile0 + t];
    }
    for (int v : seen) if (v != 1) return 4;
    printf("%lld %lld %lld %lld\n", pairs, split, nitems, singles);
    return 0;
}
"""


@pytest.fixture(scope="module")
def walker(tmp_path_factory):
    d = tmp_path_factory.mktemp("sched")
    src = d / "walk.cpp"
    src.write_text(SRC)
    exe = d / "walk"
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-I", ROOT, "-o", str(exe), str(src)])

    def run(scheme, nbh, n, d_k, sms=148):
        out = subprocess.run([str(exe), str(scheme), str(nbh), str(n), str(d_k), str(sms)], capture_output=True, text=True)
        assert out.returncode == 0, (out.returncode, scheme, nbh, n, d_k, sms)
        return tuple(int(x) for x in out.stdout.split())
    return run


FULL, SYMMETRIC, MASKED = 0, 1, 2


@pytest.mark.parametrize("scheme", [FULL, MASKED])
@pytest.mark.parametrize("nbh,n", [(1, 1), (1, 128), (3, 129), (96, 512), (96, 1024), (7, 1000), (32, 8192), (300, 384),
                                   (4096, 256), (5, 2048)])
def test_every_row_tile_is_in_exactly_one_item(walker, scheme, nbh, n):
    pairs, split, nitems, singles = walker(scheme, nbh, n, 64)
    assert nitems == split + singles and singles == 2 * (pairs - split)
    if scheme == MASKED:
        assert split == pairs           # the masked list is balanced by its longest-first order instead


def test_split_rule_cases(walker):
    # c2: 96 heads x 2 pairs on 148 CTAs: 148 pairs, then the other 44 pairs as 88 single tiles
    assert walker(FULL, 96, 512, 64) == (192, 148, 236, 88)
    # a last round that fills more than half of the CTAs stays as pairs; so does an exact multiple
    assert walker(FULL, 4096, 256, 64)[1] == 4096
    assert walker(FULL, 148, 256, 64)[1] == 148
    # fewer pairs than half of the CTAs: all single tiles
    assert walker(FULL, 8, 1024, 64) == (32, 0, 64, 64)
    # an odd number of row tiles (a pair with one tile) is never split
    assert walker(FULL, 10, 384, 64)[1] == 20
