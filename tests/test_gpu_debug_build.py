"""The -DTRJ_DEBUG build: index checks that flag, and skip, cache accesses past max_seq.

The checks live in a second library (libtrj_debug.so), so the test runs in a child process that loads that library
instead of the default one.  The bad input (an accepted path that would be compacted past the end of the cache, and a
negative path entry) is only ever given to the debug build, whose checks turn it into a flag.
"""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2406_17404_b200 import build as trj_build
import paper_2406_17404_b200 as trj
trj.use_library(trj_build.build(debug=True))
trj.lib()
out = {}
L, B, H, S, D = 2, 1, 2, 16, 64
g = torch.Generator(device="cuda"); g.manual_seed(0)
k = torch.randn(L, B, H, S, D, generator=g, device="cuda").to(torch.bfloat16)
v = torch.randn(L, B, H, S, D, generator=g, device="cuda").to(torch.bfloat16)
i32 = lambda a: torch.tensor(a, dtype=torch.int32, device="cuda")
def path(rows):
    p = np.full((1, trj.PATH_STRIDE), -1, np.int32); p[0, :len(rows)] = rows
    return torch.from_numpy(p).cuda()
# a valid call: no flag, rows moved
k0 = k.clone(); seq = i32([8])
trj.compact_rows(k, v, seq, i32([2]), path([0, 3, 5]))
out["valid_flags"] = trj.debug_flags()
out["valid_moved"] = bool(torch.equal(k[:, 0, :, 9], k0[:, 0, :, 11]) and torch.equal(k[:, 0, :, 10], k0[:, 0, :, 13]) and int(seq[0]) == 11)
# sources past the end of the 16-row cache (12 + 5 = 17) and a negative entry: flagged, those rows untouched
k1 = k.clone(); seq = i32([12])
trj.compact_rows(k, v, seq, i32([3]), path([0, 2, 5, -4]))
out["bad_flags"] = trj.debug_flags()
out["bad_rows_untouched"] = bool(torch.equal(k[:, 0, :, 14:], k1[:, 0, :, 14:]))
out["good_row_moved"] = bool(torch.equal(k[:, 0, :, 13], k1[:, 0, :, 14]))
out["flags_cleared"] = trj.debug_flags()
print(json.dumps(out))
"""


def test_debug_build_flags_and_skips_out_of_range_cache_rows():
    r = subprocess.run([sys.executable, "-c", CHILD % ROOT], capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    out = json.loads(r.stdout.strip().splitlines()[-1])
    assert out["valid_flags"] == 0 and out["valid_moved"]
    assert out["bad_flags"] == 2                            # the compaction bit, nothing else
    assert out["bad_rows_untouched"] and out["good_row_moved"]
    assert out["flags_cleared"] == 0


def test_default_build_has_no_index_checks(trj):
    with pytest.raises(trj.TrjError) as e:
        trj.debug_flags()
    assert e.value.status == 5
