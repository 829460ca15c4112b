"""The constants the paper prints (tests/golden/paper_constants.txt, each with its citation) against what the oracle
does with them: block size and rho of Eq. 1, the fixed scale s_P = 448 of Section 4.1, the 128 x 128 score tile."""
import os

import numpy as np

from oracle import mpfa_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    vals = {}
    with open(os.path.join(HERE, "golden", "paper_constants.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, value, citation = line.split(None, 2)
            assert citation.startswith("Section"), line
            vals[name] = float(value)
    return vals


def _bits(x):
    x = np.ascontiguousarray(x, np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16)


def test_block_size_and_rho_of_eq_1():
    g = _golden()
    G, rho = int(g["nvfp4_block_size"]), g["e2m1_max_magnitude"]
    assert G == 16 and orc.NBLK * G == orc.D == int(g["head_dim"])
    # one token, one head; block 3 holds one large value: only that block's scale moves, and the value that equals the
    # block's amax gets the code of rho (scale = amax / rho)
    x = np.full((1, 1, 1, 128), 0.25, np.float32)
    x[0, 0, 0, 3 * G + 5] = 3.0
    d = np.ones(1, np.float32)
    codes, sf = orc.quantize_nvfp4(_bits(x), np.zeros((1, 1, 128), np.float32), d)
    scales = np.array([orc.e4m3_decode(int(c)) for c in sf[0, 0, 0]])
    assert np.allclose(np.delete(scales, 3), 0.25 / rho, rtol=2 ** -3)        # E4M3 rounding of 0.25 / 6
    assert abs(scales[3] - 3.0 / rho) <= 2 ** -4 * 3.0 / rho
    byte = codes[0, 0, 0, (3 * G + 5) // 2]
    code = (byte >> 4) if (3 * G + 5) % 2 else (byte & 15)
    assert orc.e2m1_decode(int(code)) == rho
    assert max(orc.e2m1_decode(c) for c in range(16)) == rho


def test_fixed_scale_of_p_and_the_top_of_e4m3():
    g = _golden()
    s_p = g["p_scale"]
    assert s_p == g["e4m3_largest_normal"]
    finite = [orc.e4m3_decode(c) for c in range(0x7F)]
    assert max(finite) == s_p and orc.e4m3_decode(0x7E) == s_p
    # P = 1 (the row's arg-max key) is encoded as s_P * 1: the top code; nothing above 1 can occur, so nothing saturates
    assert orc.e4m3_encode(float(np.float32(s_p * g["p_upper_bound"]))) == 0x7E
    assert orc.e4m3_encode(float(np.float32(s_p * 0.5))) == 0x76   # 224 = 1.75 * 2^7: exactly representable, one octave down


def test_score_tile_of_the_main_loop():
    g = _golden()
    assert orc.BLOCK_KV == int(g["kv_block"]) and orc.BLOCK_KV ** 2 == int(g["scores_per_kv_block"])
