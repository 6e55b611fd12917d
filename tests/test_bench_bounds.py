"""Host arithmetic of the bench line: the algorithmic bytes, flops and exponentials of an attention call and the floors
derived from them, against figures worked out by hand for the 64K Qwen3-14B shape (B = 4, H_q = 40, H_kv = 8, d = 128,
L = 65536, T = 48: R = T G = 240 rows per KV head)."""
import importlib.util
import os

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def load_bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


class Shape:
    B, Hq, Hkv, d = 4, 40, 8, 128
    seq_len = np.full(4, 65536)


def test_kv_bytes_and_three_bounds():
    bench = load_bench()
    T = [48] * 4
    kv, qo = bench.kv_bytes(Shape, T)
    keys = 65536 + 48
    assert kv == 4 * 8 * keys * 128 * 2 * 2                    # K and V, bf16, every visible key once
    assert qo == 4 * 2 * 48 * 40 * 128 * 2                     # Q read, O written
    u = bench.three_bounds(Shape, T, 250e-6, 6447.2)
    flops = 4 * 8 * 4 * 128 * 240 * keys                       # 4 d R (L + T) per (sequence, KV head)
    exps = 4 * 8 * 240 * keys
    assert abs(u["useful_tflops"] - flops / 250e-6 / 1e12) < 1e-6
    assert abs(u["floor_us"]["hbm"] - (kv + qo) / 6447.2e9 * 1e6) < 1e-6
    assert abs(u["floor_us"]["exp"] - exps / (16 * 148 * 1.965e9) * 1e6) < 1e-6
    burst, sustained = bench.tensor_peaks_tflops()
    assert abs(u["floor_us"]["tensor"] - flops / (burst * 1e12) * 1e6) < 1e-6
    assert abs(u["frac_of_bf16_sustained"] - flops / (sustained * 1e12) / 250e-6) < 1e-9
    assert u["binding"] == max(u["floor_us"], key=u["floor_us"].get)
    assert abs(u["frac_of_binding"] - u["floor_us"][u["binding"]] / 250.0) < 1e-9
    # arithmetic intensity of the shape is R flop per KV byte
    assert abs(flops / kv - 240) < 1e-9
