"""GPU parity at the five configurations' full sizes.  Index sets, int8 codes,
scales and fp16 bits are compared bit for bit with the oracle; sums within
1e-6 of the largest magnitude.  Where the oracle's full sort of every bucket
would take minutes, a fixed subset of buckets is checked (stated per test)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_16235_b200 import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2506_16235_b200 as nsml
    from gpu_util import check_accumulate, check_compress, payload_to_device


def test_config1_single_vector():
    g = synth.config1_bucket(n=1 << 20, seed=0)
    payload, want = check_compress(g, 0.01, 8)
    assert want.k == 10486
    check_accumulate([payload], [want], g.size, zero_first=True)


@pytest.mark.parametrize("bucket", [0, 1, 2, 3])
def test_config2_resnet50_all_cases(bucket):
    g = list(synth.resnet50_buckets(seed=1))[bucket]
    assert g.size == (6_553_600 if bucket < 3 else 5_896_232)
    for ratio in (0.5, 0.1, 0.01, 0.001):
        for bits in (8, 16):
            payload, want = check_compress(g, ratio, bits)
        check_accumulate([payload], [want], g.size, zero_first=True)  # W = 1


@pytest.mark.parametrize("bucket", [0, 1, 2, 3, 4])
def test_config3_gpt2_four_workers(bucket):
    # buckets 0-1 hold the 90 %-zero embedding rows, the rest ordinary transformer layers; bucket 4 is short
    pts, pos = [], []
    n = None
    for w in range(4):
        g = synth.gpt2_bucket(bucket, seed=10 + w)
        n = g.size
        payload, want = check_compress(g, 0.01, 8)
        pts.append(payload)
        pos.append(want)
    assert n == (25_000_000 if bucket < 4 else 24_439_808) and pos[0].k == oracle.k_of(0.01, n)
    check_accumulate(pts, pos, n, zero_first=True)


def test_config4_decoder_bf16_controller_ratios():
    # one 64M-element bf16 bucket inside the layer stack, at the ratios the controller emits on the
    # 100 -> 10 -> 1 Gbps trace (first, a middle and the last one)
    bits16 = synth.decoder_bucket_bf16(5, seed=20)
    assert bits16.size == 1 << 26
    ctrl = nsml.Controller(ratio_init=0.1, ratio_min=0.001, ratio_max=0.1, startup_max_steps=0)
    ora = oracle.Controller(oracle.ControllerParams(ratio_init=0.1, ratio_min=0.001, ratio_max=0.1, startup_max_steps=0))
    dense = 2.0 * 1_315_723_264
    ratios, last = [], (0.0, 0.0)
    for step in range(90):
        r = ctrl.select_ratio(last[0], last[1], dense)
        assert r == ora.select_ratio(last[0], last[1], dense)  # every step exact
        ratios.append(r)
        sent = r * dense * 0.75
        bw = (100e9, 10e9, 1e9)[step // 30] / 8.0
        last = (sent, 1e-3 + sent / bw)
    assert ratios[0] == 0.1 and min(ratios) == 0.001
    for ratio in (ratios[0], sorted(set(ratios))[len(set(ratios)) // 2], ratios[-1]):
        check_compress(bits16, ratio, 16)
    # the last, short bucket of the set (40,654,848 elements)
    tail = synth.decoder_bucket_bf16(19, seed=20)
    assert tail.size == 1_315_723_264 - 19 * (1 << 26)
    check_compress(tail, 0.01, 16)


@pytest.mark.parametrize("ratio", [0.001, 0.05])
def test_config5_aggregation_stress(ratio):
    n, W = 350_000_000, 8
    k = oracle.k_of(ratio, n)
    pts, pos = [], []
    for w in range(W):
        idx, codes, scales = synth.stress_payload_parts(n, k, 30 + w, shared_seed=99)
        p = oracle.Payload(n=n, k=k, bits=8, idx=idx, raw=np.zeros(0, np.float32), codes=codes, scales=scales)
        pos.append(p)
        pts.append(payload_to_device(p))
    check_accumulate(pts, pos, n, zero_first=True, max_abs=127.0 * 1e-2)
