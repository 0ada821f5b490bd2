"""Prints the bandwidth of a write-then-read-back ring in device memory for a range of footprints.

    python -m paper_2405_03133_b200.probe

Each line: slot size, slots, lag (how many slots behind the writer the reader is), footprint the cache must hold
for the reads to hit = (lag + 1) * slot, and the bandwidth of write-only, read-only and write+read passes (bytes
moved over the time of the pass; write+read counts both directions).
"""
from __future__ import annotations

import torch

from . import binding as B


def main():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    buf = torch.empty((1 << 30) + 4096, dtype=torch.uint8, device=dev)
    print(f"{'slot MB':>8} {'slots':>5} {'lag':>3} {'shift':>5} {'footprint MB':>12} {'write TB/s':>10} {'read TB/s':>10} "
          f"{'write+read TB/s':>15}")
    mb = 1 << 20
    cases = []
    for slot in (4, 8, 16, 24, 32, 48, 64, 96, 128):
        cases.append((slot, 2, 1, 0))
    for slot in (8, 16, 32):
        cases.append((slot, 4, 3, 0))
    for slot in (8, 16, 32, 48):
        cases.append((slot, 2, 1, 148))  # the reader is another SM
    cases.append((256, 4, 1, 0))  # far beyond the cache: the HBM rate of the same access pattern
    for slot, slots, lag, shift in cases:
        iters = max(8, (8 << 30) // (slot * mb))
        res = []
        for mode in (1, 2, 3):
            ms = B.lory_probe_l2_ring(buf, slot * mb, slots, lag, iters, mode, shift)
            moved = iters * slot * mb * (2 if mode == 3 else 1)
            res.append(moved / (ms * 1e-3) / 1e12)
        print(f"{slot:8d} {slots:5d} {lag:3d} {shift:5d} {(lag + 1) * slot:12d} {res[0]:10.2f} {res[1]:10.2f} {res[2]:15.2f}")


if __name__ == "__main__":
    main()
