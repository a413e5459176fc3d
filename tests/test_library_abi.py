"""CPU-side checks of the C ABI: the library builds, loads, exports every declared symbol and
rejects bad parameter blocks without touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import build as rbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    rbuild.build_library()
    return rb.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rtp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rtp_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in rtp.h but not exported"
    assert set(rb.EXPORTS) == set(names)


def test_version(lib):
    assert rb.rtp_version() >= 100


def _params(**over):
    kw = dict(n_q_heads=32, n_kv_heads=8, ret_q_heads=list(range(8)), q_head_to_index_head=[0] * 4 + [1] * 4,
              index_head_kv=[0, 1], local_kv_heads=[2, 3, 4, 5, 6, 7], n_sink=4, window=2048, top_p=0.95,
              score_scale=0.125)
    kw.update(over)
    return rb.Params(**kw)


def test_workspace_bytes_and_param_validation(lib):
    good = rb.rtp_workspace_bytes(_params(), 8, 32768)
    assert good > 0 and good % 256 == 0
    assert rb.rtp_workspace_bytes(_params(), 64, 1 << 20) >= good
    assert rb.rtp_workspace_bytes(_params(top_p=0.0), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(top_p=1.5), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(top_p=float("nan")), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(n_q_heads=30), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(ret_q_heads=[0, 1, 2, 99] + [4, 5, 6, 7]), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(index_head_kv=[0, 9]), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(window=0), 8, 32768) == 0
    assert rb.rtp_workspace_bytes(_params(), 0, 32768) == 0
    p = _params()
    p.c.head_dim = 64
    assert rb.rtp_workspace_bytes(p, 8, 32768) == 0


def test_argument_blocks_have_the_library_layout(lib):
    assert lib.rtp_struct_bytes(0) == ctypes.sizeof(rb.RtpParams) > 0
    assert lib.rtp_struct_bytes(1) == ctypes.sizeof(rb.RtpCache) > 0
    assert lib.rtp_struct_bytes(2) == 0


def test_calls_without_context_are_rejected(lib):
    p = _params()
    cache = rb.RtpCache()
    assert lib.rtp_index_keys(None, p.ref(), ctypes.byref(cache), None, None, None, None, 4, None) == rb.RTP_ERR_INVALID
    assert lib.rtp_last_error(None) == b"no context"


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(rb.RtpError):
        rb.load_library(str(tmp_path / "nope.so"))
