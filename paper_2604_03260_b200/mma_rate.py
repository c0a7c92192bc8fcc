"""Table of tensor-pipe rates from the library's MMA probe (``focus_selftest_mma_rate``).

    python -m paper_2604_03260_b200.mma_rate [rounds]

One line per shape and issue pattern: cycles per round, flop per clock and SM against the nominal 8192 (dense
bf16), and TFLOP/s over the device at the clock the probe ran at.  Arithmetic on the counters only.
"""
import sys

import torch

from . import binding as fb

MODES = [  # (pair, N, ts, pattern, chains per round, label)
    (0, 128, 0, 0, 1, "1 CTA  SS M128 N128, one chain per commit (S = Q K^T as the attention kernel issues it)"),
    (0, 128, 1, 0, 1, "1 CTA  TS M128 N128, one chain per commit (O += P V)"),
    (0, 256, 0, 0, 1, "1 CTA  SS M128 N256, one chain per commit"),
    (0, 64, 0, 0, 1, "1 CTA  SS M128 N64,  one chain per commit"),
    (0, 64, 1, 0, 1, "1 CTA  TS M128 N64,  one chain per commit"),
    (1, 128, 0, 0, 1, "pair   SS M256 N128, one chain per commit"),
    (1, 256, 0, 0, 1, "pair   SS M256 N256, one chain per commit"),
    (1, 128, 1, 0, 1, "pair   TS M256 N128, one chain per commit"),
    (0, 128, 0, 1, 2, "1 CTA  two SS N128 chains per commit, alternating"),
    (0, 128, 0, 2, 2, "1 CTA  SS + TS N128 per commit, alternating"),
    (0, 128, 0, 3, 2, "1 CTA  SS then TS N128 per commit"),
    (1, 128, 0, 3, 2, "pair   SS then TS N128 per commit"),
    (0, 64, 0, 1, 2, "1 CTA  two SS N64 chains per commit, alternating"),
    (0, 64, 0, 3, 2, "1 CTA  SS then TS N64 per commit"),
]


def main(rounds=4000):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    res = torch.zeros(3, dtype=torch.int64, device="cuda")
    for pair, N, ts, pattern, chains, label in MODES:
        for _ in range(2):                       # the second launch is the one reported
            fb.focus_selftest_mma_rate(pair, N, ts, pattern, rounds, res)
            torch.cuda.synchronize()
        cycles, ns, fault = (int(x) for x in res.tolist())
        flop_sm = chains * 2.0 * 128 * N * 128 * rounds           # per SM (a pair does 256 rows on two SMs)
        print(f"{label:<92s} fault {fault}  cycles/round {cycles / rounds:7.1f}  flop/clk/SM {flop_sm / cycles:6.0f} "
              f"({flop_sm / cycles / 8192:.2f} of 8192)  {flop_sm * sms / (ns * 1e-9) / 1e12:5.0f} TFLOP/s at {cycles / (ns * 1e-3):.0f} MHz")


if __name__ == "__main__":
    main(int(sys.argv[1]) if len(sys.argv) > 1 else 4000)
