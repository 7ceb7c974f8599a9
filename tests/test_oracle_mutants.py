"""The pins must be able to fail: plant plausible mistakes in a COPY of the oracle's C source
(on the CPU, never in the product) and check that the pin checks reject every one of them."""
import ctypes
import math
import os
import subprocess

import numpy as np
import pytest

from oracle import attention as oa
from paper_2605_23296_b200 import workloads as wl

SRC = os.path.join(os.path.dirname(oa.__file__), "attn_oracle.c")

MUTANTS = {
    # name: (text in the source, replacement)
    "strict_causal_mask": ("attend_row(q_row, kb, vb, i + 1,", "attend_row(q_row, kb, vb, i > 0 ? i : 1,"),
    "scale_dropped": ("        s *= scale;\n", ""),
    "head_map_modulo": ("J->Hkv, h / G, J->d", "J->Hkv, h % J->Hkv, J->d"),
    "no_max_subtraction_sign": ("scratch[j] = exp(scratch[j] - m);", "scratch[j] = exp(m - scratch[j]);"),
    "denominator_off_by_one_term": ("    for (int c = 0; c < d; ++c) out[c] /= denom;", "    for (int c = 0; c < d; ++c) out[c] /= (denom + 1.0);"),
    "value_head_zero": ("const uint16_t* vj = v + j * stride + (int64_t)g * d;", "const uint16_t* vj = v + j * stride;"),
    "block_offset_ignored": ("const uint16_t* kb = J->k + start * (int64_t)J->Hkv * J->d;", "const uint16_t* kb = J->k;"),
}


def _bf(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _prefill(lib, q, k, v, cu, scale):
    tokens, Hq, d = q.shape
    Hkv = k.shape[1]
    cu = np.ascontiguousarray(cu, dtype=np.int32)
    out = np.empty((tokens, Hq, d), dtype=np.float64)
    u16p, f64p = ctypes.POINTER(ctypes.c_uint16), ctypes.POINTER(ctypes.c_double)
    lib.oracle_prefill.restype = ctypes.c_int
    rc = lib.oracle_prefill(
        np.ascontiguousarray(q).ctypes.data_as(u16p), np.ascontiguousarray(k).ctypes.data_as(u16p),
        np.ascontiguousarray(v).ctypes.data_as(u16p), cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
        ctypes.c_int(len(cu) - 1), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_double(scale),
        None, ctypes.c_int64(tokens), out.ctypes.data_as(f64p), ctypes.c_int(1))
    assert rc == 0
    return out


def pins_hold(lib) -> bool:
    """A condensed set of the pins of test_oracle_pins.py, evaluated on `lib`."""
    rng = np.random.default_rng(0)
    try:
        # two-key closed form, with a scale that matters
        q = _bf([[[2.0, 0.0]], [[2.0, 0.0]]]); k = _bf([[[0.0, 5.0]], [[1.0, -3.0]]]); v = _bf([[[1.0, -2.0]], [[3.0, 4.0]]])
        out = _prefill(lib, q, k, v, [0, 2], 0.5)
        w1 = math.e / (1.0 + math.e)
        if not np.allclose(out[1, 0], [1 + 2 * w1, -2 + 6 * w1], rtol=1e-13) or not np.array_equal(out[0, 0], [1.0, -2.0]):
            return False
        # K = 0: running mean; V constant per kv head identifies the head map (Hq=6, Hkv=3)
        L = 9
        qq = _bf(rng.standard_normal((L, 6, 4), dtype=np.float32)); kk = np.zeros((L, 3, 4), dtype=np.uint16)
        vv = _bf(np.broadcast_to(np.arange(3, dtype=np.float32)[None, :, None], (L, 3, 4)))
        out = _prefill(lib, qq, kk, vv, [0, L], 1.0)
        if not all(np.allclose(out[:, h], h // 2, atol=1e-14) for h in range(6)):
            return False
        # two blocks: the batch equals each block alone, and large scores do not overflow
        L1, L2 = 7, 5
        qq = _bf(20 * rng.standard_normal((L1 + L2, 2, 8), dtype=np.float32))
        kk = _bf(20 * rng.standard_normal((L1 + L2, 1, 8), dtype=np.float32))
        vv = _bf(rng.standard_normal((L1 + L2, 1, 8), dtype=np.float32))
        both = _prefill(lib, qq, kk, vv, [0, L1, L1 + L2], 0.5)
        alone = _prefill(lib, qq[L1:], kk[L1:], vv[L1:], [0, L2], 0.5)
        if not np.isfinite(both).all() or not np.array_equal(both[L1:], alone):
            return False
        # against an independent dense evaluation
        qf, kf, vf = (oa.bf16_bits_to_f64(t) for t in (qq[:L1], kk[:L1], vv[:L1]))
        s = np.einsum("ihc,jc->hij", qf, kf[:, 0]) * 0.5
        s = np.where(np.triu(np.ones((L1, L1), bool), 1)[None], -np.inf, s)
        p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
        ref = np.einsum("hij,jc->ihc", p, vf[:, 0])
        return bool(np.allclose(both[:L1], ref, rtol=1e-10, atol=1e-12))
    except Exception:
        return False


def _compile(text: str, tmp_path, name: str):
    src = tmp_path / f"{name}.c"
    lib = tmp_path / f"lib{name}.so"
    src.write_text(text)
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-o", str(lib), str(src), "-lm", "-lpthread"], check=True)
    return ctypes.CDLL(str(lib))


def test_unmodified_copy_passes(tmp_path):
    assert pins_hold(_compile(open(SRC).read(), tmp_path, "clean"))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    assert not pins_hold(_compile(text.replace(old, new), tmp_path, name))
