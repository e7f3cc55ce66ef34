"""nsml_select_ratio (host C++) against the oracle controller: bit-identical
doubles on seeded link traces, plus argument handling and checkpointing."""
import math

import numpy as np
import pytest

from oracle import Controller as OracleController, ControllerParams
from conftest import read_golden
from paper_2506_16235_b200 import build as nsml_build

nsml_build.build()
import paper_2506_16235_b200 as nsml  # noqa: E402


def link_trace(seed, steps, dense, bw_steps, jitter=0.02):
    """Transfer time of `nbytes` on a link: rtprop0 + nbytes/BW(step), BW a
    step function, with a seeded +-2 % jitter."""
    rng = np.random.default_rng(seed)
    rt0 = 1e-3
    for s in range(steps):
        bw = bw_steps[min(len(bw_steps) - 1, s * len(bw_steps) // steps)]
        yield bw, rt0, 1.0 + jitter * (2.0 * rng.random() - 1.0)


PARAM_SETS = [
    {},
    {"btlbw_window": 0, "rtprop_window": 0},
    {"startup_max_steps": 0, "ratio_init": 0.1, "ratio_min": 0.001},
    {"beta1": 0.25, "startup_max_steps": 3, "rtt_excess": 2.0, "btlbw_window": 3, "rtprop_window": 7},
    {"alpha": 0.7, "beta2": 0.003, "bdp_frac": 0.8},
]


@pytest.mark.parametrize("overrides", PARAM_SETS)
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_matches_oracle_bit_for_bit(overrides, seed):
    dense = 1.315723264e9 * 2  # bytes of a bf16 1.3B-parameter gradient set
    lib_c = nsml.Controller(**overrides)
    ora_c = OracleController(ControllerParams(**overrides))
    r_lib = lib_c.select_ratio(0, 0, dense)
    r_ora = ora_c.select_ratio(0, 0, dense)
    assert r_lib == r_ora
    for bw_gbps, rt0, jit in link_trace(seed, 120, dense, (100, 10, 1)):
        nbytes = r_ora * dense * 0.75  # about 6 bytes per kept fp16 entry vs 8 dense
        secs = (rt0 + nbytes / (bw_gbps * 1e9 / 8)) * jit
        r_lib = lib_c.select_ratio(nbytes, secs, dense)
        r_ora = ora_c.select_ratio(nbytes, secs, dense)
        assert r_lib == r_ora  # exact doubles
        st = lib_c.state()
        assert (st.ebb, st.btlbw, st.rtprop, st.bdp) == (ora_c.last_ebb, ora_c.btlbw, ora_c.rtprop, ora_c.bdp)
        assert st.phase == ora_c.phase and st.calls == ora_c.calls


def test_golden_startup_cap_exit_through_the_library():
    gold = read_golden("h7_startup_cap.txt")
    kv = dict(item.split("=") for item in gold["params"][0])
    c = nsml.Controller(ratio_init=float(kv["ratio_init"]), beta1=float(kv["beta1"]), ratio_max=float(kv["ratio_max"]),
                        startup_max_steps=int(kv["startup_max_steps"]))
    dense = float(kv["next_dense_bytes"])
    assert c.select_ratio(0, 0, dense) == float(kv["ratio_init"])
    for row in gold["step"]:
        got = c.select_ratio(float(row[0]), float(row[1]), dense)
        st = c.state()
        assert (st.phase, st.startup_steps) == (int(row[2]), int(row[3]))
        assert got == float(row[4])


def test_golden_trace_through_the_library():
    gold = read_golden("h4_controller.txt")
    kv = dict(item.split("=") for item in gold["params"][0])
    c = nsml.Controller(ratio_init=float(kv["ratio_init"]), startup_max_steps=int(kv["startup_max_steps"]),
                        btlbw_window=int(kv["btlbw_window"]), rtprop_window=int(kv["rtprop_window"]))
    dense = float(kv["next_dense_bytes"])
    assert c.select_ratio(0, 0, dense) == float(kv["ratio_init"])
    for row in gold["step"]:
        nbytes, secs, ebb, btlbw, rtprop, bdp, ratio = (float(x) for x in row)
        assert c.select_ratio(nbytes, secs, dense) == ratio
        st = c.state()
        assert (st.ebb, st.btlbw, st.rtprop, st.bdp) == (ebb, btlbw, rtprop, bdp)


def test_adapts_to_bandwidth_drop_only_with_windows():
    dense = 2.6e9

    def run(**kw):
        c = nsml.Controller(ratio_init=0.1, ratio_min=0.001, startup_max_steps=0, **kw)
        r = c.select_ratio(0, 0, dense)
        out = []
        for bw_gbps, rt0, _ in link_trace(0, 300, dense, (100, 10, 1), jitter=0.0):
            nbytes = r * dense
            r = c.select_ratio(nbytes, rt0 + nbytes / (bw_gbps * 1e9 / 8), dense)
            out.append(r)
        return out

    win = run()
    lit = run(btlbw_window=0, rtprop_window=0)
    # with sliding windows the mean ratio falls with the link; plateau means ordered
    m = [float(np.mean(win[a:b])) for a, b in ((50, 100), (150, 200), (250, 300))]
    assert m[0] > 3 * m[1] > 9 * m[2] / 1.5
    # the literal all-time max keeps BDP at its historic high: ratio never comes down
    assert np.mean(lit[250:300]) > 5 * np.mean(win[250:300])


def test_rejects_bad_arguments_and_keeps_state():
    c = nsml.Controller(startup_max_steps=0, ratio_init=0.3)
    c.select_ratio(0, 0, 1e6)
    c.select_ratio(1e6, 1.0, 1e6)
    before = c.save()
    for args in ((1e6, 0.0, 1e6), (1e6, -1.0, 1e6), (1e6, math.nan, 1e6), (-1.0, 1.0, 1e6),
                 (math.inf, 1.0, 1e6), (1e6, 1.0, math.nan), (1e6, 1.0, -5.0)):
        with pytest.raises(nsml.NsmlError) as e:
            c.select_ratio(*args)
        assert e.value.status == nsml.NSML_ERR_ARG
    assert c.save() == before
    for bad in ({"alpha": 1.5}, {"ratio_min": 0.0}, {"ratio_init": 2.0}, {"beta2": -1.0}, {"btlbw_window": -1},
                {"rtprop_window": 5000}, {"rtt_excess": 0.5}):
        with pytest.raises(nsml.NsmlError):
            nsml.Controller(**bad)


def test_checkpoint_resume_continues_identically():
    dense = 1e9
    a = nsml.Controller(btlbw_window=4, rtprop_window=6)
    r = a.select_ratio(0, 0, dense)
    trace = list(link_trace(3, 80, dense, (40, 4)))
    for bw, rt0, jit in trace[:37]:
        r = a.select_ratio(r * dense, (rt0 + r * dense / (bw * 1e9 / 8)) * jit, dense)
    blob = a.save()
    b = nsml.Controller()  # other parameters: load replaces them
    b.load(blob)
    ra = rb = r
    for bw, rt0, jit in trace[37:]:
        ra = a.select_ratio(ra * dense, (rt0 + ra * dense / (bw * 1e9 / 8)) * jit, dense)
        rb = b.select_ratio(rb * dense, (rt0 + rb * dense / (bw * 1e9 / 8)) * jit, dense)
        assert ra == rb
    with pytest.raises(nsml.NsmlError):
        b.load(blob[:-8])
    with pytest.raises(nsml.NsmlError):
        b.load(b"\0" * len(blob))
