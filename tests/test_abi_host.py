"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header
declares, and its pure host functions behave as documented."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "bigcn.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2210_13149_b200 import build
    build.build()
    from paper_2210_13149_b200 import binding
    return binding.load()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bigcn_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_core_calls():
    names = declared_functions()
    for core in ("bigcn_pack_features", "bigcn_pack_weights", "bigcn_layer_forward", "bigcn_forward"):
        assert core in names


def test_library_exports_every_declared_symbol(lib):
    from paper_2210_13149_b200 import binding
    names = declared_functions()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
        assert name in binding.SIGNATURES, "binding lacks a prototype for %s" % name
    assert sorted(binding.SIGNATURES) == names


def test_packed_stride_words(lib):
    f = lib.bigcn_packed_stride_words
    assert [f(d) for d in (1, 32, 33, 100, 128, 129, 256, 602, 1433, 3703)] == [4, 4, 4, 4, 4, 8, 8, 20, 48, 116]
    assert f(0) == 0 and f(-5) == 0


def test_status_strings(lib):
    seen = {lib.bigcn_status_string(s) for s in range(9)}
    assert len(seen) == 9 and b"ok" in seen


def test_workspace_bytes_grows_with_the_problem(lib):
    def ws(n, dims, host_io=0):
        arr = (ctypes.c_int32 * len(dims))(*dims)
        return lib.bigcn_workspace_bytes(n, 10 * n, arr, len(dims) - 1, host_io)
    small = ws(1000, [100, 64, 7])
    big = ws(100000, [100, 64, 7])
    assert 0 < small < big
    # the zeta scratch of the widest layer (fp32) must fit
    assert ws(1000, [100, 256, 7]) >= 1000 * 256 * 4
    assert ws(100000, [100, 64, 7], 1) >= big + 100000 * 100 * 4    # staging for X (and logits)
    assert ws(1000, [100, 0, 7]) == 0            # invalid widths
    assert ws(-1, [100, 64, 7]) == 0


def test_create_fails_loudly_without_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    st = lib.bigcn_create(ctypes.byref(h), 0, None)
    assert st != 0 and not h.value
    from paper_2210_13149_b200 import binding
    with pytest.raises(RuntimeError):
        binding.BiGCN(0)


def test_null_context_is_rejected(lib):
    assert lib.bigcn_set_workspace(None, None, 0) != 0
    assert lib.bigcn_sync_check(None) != 0
    assert lib.bigcn_launch_count(None) == 0
    assert lib.bigcn_last_error(None) == b"context is null"


def test_layer_width_limits_are_refused_on_the_host(lib):
    """A layer wider than the contraction kernels serve (their shared-memory tiles hold the whole packed K extent)
    is refused as unsupported by argument validation, before any GPU work: checked through the entry point that needs
    no context.  The header states the limits."""
    from paper_2210_13149_b200 import binding
    text = open(HEADER).read()
    max_in = int(re.search(r"#define BIGCN_MAX_D_IN (\d+)", text).group(1))
    max_out = int(re.search(r"#define BIGCN_MAX_D_OUT (\d+)", text).group(1))
    assert max_in * 384 // 32 + 1024 <= 200 * 1024          # 96 words of tile and panel per 32 inputs + slack fit the kernel's shared memory
    g = binding.bigcn_graph(n=4, nnz=4, rowptr=None, colidx=None, val=None, dinv=None)
    fake = ctypes.c_void_p(256)                             # never dereferenced: validation fails first

    def call(d_in, d_out):
        layer = binding.bigcn_layer(d_in=d_in, d_out=d_out, w_bitsT=fake, alpha=fake, in_shift=None, in_scale=None)
        return lib.bigcn_layer_forward_noalloc(None, ctypes.byref(g), ctypes.byref(layer), fake, fake, fake, d_out, None, None, None)

    assert call(max_in + 1, 8) == 7                         # BIGCN_ERR_UNSUPPORTED
    assert call(8, max_out + 1) == 7
    assert call(0, 8) == 2                                  # BIGCN_ERR_SHAPE
    assert call(max_in, max_out) == 1                       # passes the width checks; the null rowptr is caught next
