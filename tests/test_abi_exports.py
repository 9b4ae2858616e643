"""The C-ABI library loads without a GPU and exports every symbol include/tng.h declares."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def declared_symbols():
    text = (ROOT / "include" / "tng.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tng_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_1901_08227_b200 import build
    return ctypes.CDLL(str(build.build()))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "tng_step" in names and "tng_create" in names and len(names) >= 20
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing


def test_binding_lists_the_same_symbols():
    from paper_1901_08227_b200 import tng
    assert sorted(tng.EXPORTS) == declared_symbols()


def test_host_only_calls_work_without_a_device():
    from paper_1901_08227_b200 import tng
    ctx = tng.Context(1000, 4, 1, tng.CODEC_TERN2, tng.NORM_DIFF, block=0)
    st = ctx.stats()
    assert st.d == 1000 and st.M == 4 and st.k == 0 and st.rounds == 0
    assert st.bits_per_coord == pytest.approx(2 + 32 / 1000 + 64 / 1000)
    assert ctx.workspace_bytes() > 1000 * 4 * 2
    with pytest.raises(tng.TngError) as e:
        ctx.set_option("block", 256)                    # sized already: options are frozen
    assert e.value.status == tng.ERR_STATE
    ctx.close()
    for bad in [dict(d=0, M=1, K=1), dict(d=8, M=0, K=1), dict(d=8, M=65, K=1), dict(d=8, M=1, K=17)]:
        with pytest.raises(tng.TngError) as e:
            tng.Context(bad["d"], bad["M"], bad["K"], tng.CODEC_TERN2, tng.NORM_DIFF)
        assert e.value.status == tng.ERR_INVALID_ARG
    with pytest.raises(tng.TngError):
        tng.Context(8, 1, 1, 3, tng.NORM_DIFF)
    with pytest.raises(tng.TngError):
        tng.Context(8, 1, 1, tng.CODEC_TERN2, tng.NORM_DIFF, block=100)
    with pytest.raises(tng.TngError):
        tng.Context(8, 1, 1, tng.CODEC_QSGD4, tng.NORM_DIFF, qsgd_levels=8)
    assert tng.status_string(tng.ERR_NONFINITE) == "non-finite block scale"
