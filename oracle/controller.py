"""Oracle for the network-sensing ratio controller (Alg. 1, Eq. 1-3).

TEST INFRASTRUCTURE ONLY (see the package docstring).

One call per gradient-transmission interval.  The call for interval i is
given the size and the measured transfer time of interval i-1 and the size
the next transfer would have at ratio 1; it returns the ratio (kept fraction)
to compress interval i with.  All arithmetic is IEEE double, each formula in
the operand order the paper prints it.

NetSense phase (Alg. 1 Step 2):
    EBB    = data_size_{i-1} / RTT_{i-1}                       (Eq. 1)
    BtlBw  = max of the EBB samples, RTprop = min of the RTT samples
    BDP    = BtlBw * RTprop                                    (Eq. 2)
    ratio  = max(ratio_min, ratio * alpha)   if data_size > bdp_frac * BDP
           = min(ratio_max, ratio + beta2)   otherwise         (Eq. 3)

Readings where the paper is silent:
  * data_size in Eq. 3 is the size of the upcoming transfer at the current
    ratio, ratio * next_dense_bytes (BDP is estimated "prior to each data
    transmission").
  * "maximum observed" / "minimum recorded" run over the last btlbw_window /
    rtprop_window samples; window 0 is the literal all-time extreme.
  * Start-up (Alg. 1 Step 1): the first call returns ratio_init.  Each later
    start-up call records the sample, then leaves start-up if the measured
    time exceeds rtt_excess * RTprop, or startup_max_steps increments were
    made, or the ratio reached ratio_max; otherwise ratio += beta1 (capped).
    The call that leaves start-up applies the NetSense rule at once.
    beta1, startup_max_steps and rtt_excess are not in the paper.
  * A non-positive or non-finite transfer time, or a negative or non-finite
    size, is rejected (ValueError) and leaves the state untouched.
"""
from __future__ import annotations

import math
from collections import deque
from dataclasses import dataclass


@dataclass
class ControllerParams:
    ratio_init: float = 0.01  # Alg. 1 Step 1
    ratio_min: float = 0.005  # Eq. 3
    ratio_max: float = 1.0  # Eq. 3
    alpha: float = 0.5  # Section 4.1
    beta1: float = 0.1  # not given in the paper
    beta2: float = 0.01  # Section 4.1
    bdp_frac: float = 0.9  # Eq. 3
    startup_max_steps: int = 10  # not given ("first few steps")
    rtt_excess: float = 1.25  # not given ("excessive RTT")
    btlbw_window: int = 10  # 0 = all-time maximum (literal reading)
    rtprop_window: int = 100  # 0 = all-time minimum (literal reading)


class Controller:
    STARTUP = 0
    NETSENSE = 1

    def __init__(self, params: ControllerParams | None = None):
        self.p = params or ControllerParams()
        self.ratio = float(self.p.ratio_init)
        self.phase = self.STARTUP if self.p.startup_max_steps > 0 else self.NETSENSE
        self.calls = 0
        self.startup_steps = 0
        self.ebb_samples = deque()
        self.rtt_samples = deque()
        self.btlbw = 0.0
        self.rtprop = math.inf
        self.bdp = 0.0
        self.last_ebb = 0.0

    def _record(self, nbytes: float, seconds: float) -> None:
        ebb = nbytes / seconds  # Eq. 1
        self.last_ebb = ebb
        self.ebb_samples.append(ebb)
        self.rtt_samples.append(seconds)
        if self.p.btlbw_window > 0:
            while len(self.ebb_samples) > self.p.btlbw_window:
                self.ebb_samples.popleft()
            self.btlbw = max(self.ebb_samples)
        else:
            self.btlbw = max(self.btlbw, ebb)
            self.ebb_samples.clear()
        if self.p.rtprop_window > 0:
            while len(self.rtt_samples) > self.p.rtprop_window:
                self.rtt_samples.popleft()
            self.rtprop = min(self.rtt_samples)
        else:
            self.rtprop = min(self.rtprop, seconds)
            self.rtt_samples.clear()
        self.bdp = self.btlbw * self.rtprop  # Eq. 2

    def _netsense_adjust(self, next_dense_bytes: float) -> None:
        data_size = self.ratio * next_dense_bytes
        if data_size > self.p.bdp_frac * self.bdp:  # Eq. 3, congested branch
            self.ratio = max(self.p.ratio_min, self.ratio * self.p.alpha)
        else:  # Eq. 3, probing branch
            self.ratio = min(self.p.ratio_max, self.ratio + self.p.beta2)

    def select_ratio(self, last_bytes: float, last_seconds: float, next_dense_bytes: float) -> float:
        last_bytes = float(last_bytes)
        last_seconds = float(last_seconds)
        next_dense_bytes = float(next_dense_bytes)
        if self.calls == 0:
            # nothing has been sent yet: the measurement arguments are ignored
            if not (math.isfinite(next_dense_bytes) and next_dense_bytes >= 0.0):
                raise ValueError("next_dense_bytes must be finite and >= 0")
            self.calls = 1
            return self.ratio
        ok = (
            math.isfinite(last_bytes) and last_bytes >= 0.0
            and math.isfinite(last_seconds) and last_seconds > 0.0
            and math.isfinite(next_dense_bytes) and next_dense_bytes >= 0.0
        )
        if not ok:
            raise ValueError("bad measurement")
        self.calls += 1
        self._record(last_bytes, last_seconds)
        if self.phase == self.STARTUP:
            leave = (
                last_seconds > self.p.rtt_excess * self.rtprop
                or self.startup_steps >= self.p.startup_max_steps
                or self.ratio >= self.p.ratio_max
            )
            if not leave:
                self.ratio = min(self.p.ratio_max, self.ratio + self.p.beta1)
                self.startup_steps += 1
                return self.ratio
            self.phase = self.NETSENSE
        self._netsense_adjust(next_dense_bytes)
        return self.ratio
