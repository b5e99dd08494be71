import numpy as np
import pytest

from paper_2411_03786_b200.tablefile import load_table, save_table


def test_roundtrip_and_damage_detection(tmp_path):
    g = np.random.default_rng(0)
    tab = g.integers(0, 50, (50, 4)).astype(np.int32)
    ext = g.integers(0, 50, (50, 4, 3)).astype(np.int32)
    p = str(tmp_path / "t.ngtab")
    save_table(p, tab, ext, d=64, meta={"seed": 1})
    t2, e2, h = load_table(p)
    assert np.array_equal(t2, tab) and np.array_equal(e2, ext) and h["d"] == 64 and h["meta"] == {"seed": 1}
    save_table(p, tab)
    t3, e3, _ = load_table(p)
    assert np.array_equal(t3, tab) and e3 is None
    blob = bytearray(open(p, "rb").read())
    blob[-1] ^= 1
    open(p, "wb").write(bytes(blob))
    with pytest.raises(ValueError):
        load_table(p)
    open(p, "wb").write(b"something else")
    with pytest.raises(ValueError):
        load_table(p)
