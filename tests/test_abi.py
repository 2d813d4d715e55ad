"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments on the host.
No kernel is launched here; these run without a GPU."""
import ctypes
import math
import os
import re

import pytest

from paper_2609_16874_b200 import binding as cb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cpe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cpe_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = cb.load()
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in cpe.h but not exported by libcpe.so"
    assert sorted(cb.EXPORTS) == names, "binding.EXPORTS and cpe.h disagree"
    for n in names:
        assert hasattr(cb, n), f"binding lacks a function named {n}"


def test_params_struct_and_workspace_size():
    p = cb.make_params(cb.CPE_F16, 256, 128, flags=cb.CPE_FLAG_NO_PRUNE)
    assert p.struct_size == ctypes.sizeof(cb.cpe_params) == 56
    n = cb.cpe_workspace_size(1, 1024, 2048, 8, p)
    # votes 128 KB + peak embeddings 1024*32*4 + palettes + lists: a few hundred KB, far below one plane
    assert 128 * 1024 * 4 // 4 <= n < 2 * 1024 * 1024
    assert n % 256 == 0
    # the pruned assignment (default) adds each pixel's bin (4 bytes per pixel), two queues for a quarter of the pixels each,
    # the per-bin sums and the candidate lists
    pp = cb.make_params(cb.CPE_F16, 256, 128)
    n_pruned = cb.cpe_workspace_size(1, 1024, 2048, 8, pp)
    assert n + 6 * 1024 * 2048 <= n_pruned < n + 6 * 1024 * 2048 + 4 * 1024 * 1024
    # ... but not when no image can have more peaks than the all-pairs kernel takes, nor on small inputs
    assert cb.cpe_workspace_size(1, 512, 512, 8, pp) < 4 * 512 * 512
    assert cb.cpe_workspace_size(1, 1024, 2048, 8, cb.make_params(cb.CPE_F16, 256, 128, max_instances=32)) < n
    p2 = cb.make_params(cb.CPE_F16, 256, 128, flags=cb.CPE_FLAG_WRITE_SCORES | cb.CPE_FLAG_NO_PRUNE)
    assert cb.cpe_workspace_size(1, 1024, 2048, 8, p2) >= n + 2 * 4 * 1024 * 2048
    assert cb.cpe_workspace_size(0, 4, 4, 4, p) == 0
    assert cb.cpe_workspace_size(1, 4, 4, 17, p) == 0
    bad = cb.make_params(cb.CPE_F16, 5000, 8)
    assert cb.cpe_workspace_size(1, 4, 4, 4, bad) == 0


def test_argument_errors_are_reported_before_any_launch():
    p = cb.make_params(cb.CPE_F32, 32, 32)
    p.workspace = 256 * 1000
    p.workspace_bytes = 1 << 30
    fake = 4096
    assert cb.cpe_decode(0, 0, 0, 1, 8, 8, 4, p, fake, fake, fake) == cb.CPE_ERR_NULL
    assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 4, p, 0, fake, fake) == cb.CPE_ERR_NULL
    assert cb.cpe_decode(0, fake, 0, 0, 8, 8, 4, p, fake, fake, fake) == cb.CPE_ERR_SIZE
    assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 0, p, fake, fake, fake) == cb.CPE_ERR_SIZE
    assert cb.cpe_decode(0, fake + 2, 0, 1, 8, 8, 4, p, fake, fake, fake) == cb.CPE_ERR_ALIGN
    small = cb.make_params(cb.CPE_F32, 32, 32, workspace=256 * 1000, workspace_bytes=128)
    assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 4, small, fake, fake, fake) == cb.CPE_ERR_WORKSPACE
    mis = cb.make_params(cb.CPE_F32, 32, 32, workspace=256 * 1000 + 8, workspace_bytes=1 << 30)
    assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 4, mis, fake, fake, fake) == cb.CPE_ERR_WORKSPACE
    for kw, code in [(dict(vote_threshold=-1), cb.CPE_ERR_PARAM), (dict(max_instances=0), cb.CPE_ERR_PARAM),
                     (dict(levels=-2), cb.CPE_ERR_PARAM), (dict(tau=math.nan), cb.CPE_ERR_PARAM),
                     (dict(flags=cb.CPE_FLAG_SOFT_VOTE, soft_threshold=-1.0), cb.CPE_ERR_PARAM),
                     (dict(flags=cb.CPE_FLAG_SOFT_VOTE, soft_threshold=math.inf), cb.CPE_ERR_PARAM),
                     (dict(flags=cb.CPE_FLAG_SOFT_VOTE, soft_threshold=math.nan), cb.CPE_ERR_PARAM),
                     (dict(flags=cb.CPE_FLAG_SOFT_VOTE | cb.CPE_FLAG_REFINE, soft_threshold=1.0), cb.CPE_ERR_PARAM)]:
        q = cb.make_params(cb.CPE_F32, 32, 32, workspace=256 * 1000, workspace_bytes=1 << 30, **kw)
        assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 4, q, fake, fake, fake) == code
    q = cb.make_params(7, 32, 32, workspace=256 * 1000, workspace_bytes=1 << 30)
    assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 4, q, fake, fake, fake) == cb.CPE_ERR_DTYPE
    q = cb.make_params(cb.CPE_F32, 32, 32, workspace=256 * 1000, workspace_bytes=1 << 30)
    q.struct_size = 12
    assert cb.cpe_decode(0, fake, 0, 1, 8, 8, 4, q, fake, fake, fake) == cb.CPE_ERR_PARAM


def test_intermediate_addresses_are_inside_the_workspace_and_disjoint():
    p = cb.make_params(cb.CPE_F32, 64, 48, flags=cb.CPE_FLAG_WRITE_SCORES | cb.CPE_FLAG_KEEP_VOTES, max_instances=100)
    base = 1 << 20
    p.workspace = base
    p.workspace_bytes = cb.cpe_workspace_size(2, 30, 50, 8, p)
    spans = []
    for which in range(10):
        rc, ptr, size = cb.cpe_get_intermediate(p, which, 2, 30, 50, 8)
        assert rc == cb.CPE_OK and size > 0
        assert base <= ptr and ptr + size <= base + p.workspace_bytes and ptr % 256 == 0
        spans.append((ptr, ptr + size))
    spans.sort()
    for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
        assert a1 <= b0
    rc, ptr, size = cb.cpe_get_intermediate(p, cb.CPE_INT_VOTES, 2, 30, 50, 8)
    assert size == 2 * 64 * 48 * 4
    assert cb.cpe_get_intermediate(p, 99, 2, 30, 50, 8)[0] == cb.CPE_ERR_WHICH
    p.flags = 0
    assert cb.cpe_get_intermediate(p, cb.CPE_INT_BEST_SCORE, 2, 30, 50, 8)[0] == cb.CPE_ERR_WHICH
    assert cb.cpe_get_intermediate(p, cb.CPE_INT_VOTES, 2, 30, 50, 8)[0] == cb.CPE_ERR_WHICH


def test_strerror_covers_every_code():
    seen = set()
    for code in range(0, -12, -1):
        s = cb.cpe_strerror(code)
        assert s and s != "unknown error code"
        seen.add(s)
    assert len(seen) == 12
    assert cb.cpe_strerror(-99) == "unknown error code"
    assert cb.cpe_graph_launch(0, 0) == cb.CPE_ERR_NULL
    assert cb.cpe_graph_kernel_nodes(0) == 0
