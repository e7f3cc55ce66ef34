"""GPU parity at the five configurations' full sizes.  Index sets, int8 codes,
scales and fp16 bits are compared bit for bit with the oracle; sums within
1e-6 of the largest magnitude."""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2506_16235_b200 as nsml
    from gpu_util import assert_payload_equal, check_accumulate, check_compress, payload_to_device, to_device_grad


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


DECODER_ELEMS = 1_315_723_264
# steps of the 90-step link trace whose ratios are compressed with: the start, the descent and the
# oscillation on the 100 Gbps plateau, the 10 Gbps plateau, and the floor reached on the 1 Gbps plateau
CONFIG4_STEPS = (0, 1, 5, 31, 41, 60, 89)


def config4_trace():
    """Ratios the controller emits on the 100 -> 10 -> 1 Gbps step trace (30 steps per plateau), every
    step compared with the oracle's controller."""
    ctrl = nsml.Controller(ratio_init=0.1, ratio_min=0.001, ratio_max=0.1, startup_max_steps=0)
    ora = oracle.Controller(oracle.ControllerParams(ratio_init=0.1, ratio_min=0.001, ratio_max=0.1, startup_max_steps=0))
    dense = 2.0 * DECODER_ELEMS
    ratios, last = [], (0.0, 0.0)
    for step in range(90):
        r = ctrl.select_ratio(last[0], last[1], dense)
        assert r == ora.select_ratio(last[0], last[1], dense)  # every step exact
        ratios.append(r)
        sent = r * dense * 0.75
        bw = (100e9, 10e9, 1e9)[step // 30] / 8.0
        last = (sent, 1e-3 + sent / bw)
    assert ratios[0] == 0.1 and min(ratios) == 0.001
    return ratios


@pytest.mark.parametrize("bucket", range(20))
def test_config4_decoder_bf16_every_bucket_at_controller_ratios(bucket):
    # every 64M-element bf16 bucket of the 1.3B-parameter set (the last one is short), fp16 values, at six
    # distinct ratios the controller emits across the three plateaus of the link trace
    ratios = config4_trace()
    picked = sorted({ratios[s] for s in CONFIG4_STEPS}, reverse=True)
    assert len(picked) >= 6 and picked[0] == 0.1 and picked[-1] == 0.001
    bits16 = synth.decoder_bucket_bf16(bucket, seed=20)
    assert bits16.size == ((1 << 26) if bucket < 19 else DECODER_ELEMS - 19 * (1 << 26))
    wants = oracle.compress_many(oracle.widen_bf16(bits16), picked, 16)
    grad = to_device_grad(bits16)
    n = grad.numel()
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(n, nsml.NSML_BF16), "cuda")
    for ratio, want in zip(picked, wants):
        payload = nsml.nsml_compress(grad, ratio, 16, workspace=ws)
        status = nsml.nsml_last_status(ws)
        assert status == 0, nsml.nsml_strerror(status)
        assert_payload_equal(payload, want)


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
