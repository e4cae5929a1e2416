"""Oracle: the hardware cost model behind the paper's energy and speed-up figures (Section 5, System
Implementation; used in Section 6.3).  Test infrastructure only.

What the paper fixes (Section 5): an XPU with 16.4 TOPS at 3.18 TOPS/W; LPDDR4 DRAM with about 104 Gbps and up to
1.5 pJ/bit per read or write; UFS 3.1 Flash with 10 Gbps and 103 pJ/bit, holding all weights and touched only when
a slice misses in DRAM.

The paper never writes the model out.  Readings (stated once, used by this oracle and the host code alike):
  * a step's quantities are the bytes fetched from Flash (misses), the bytes the computation reads from DRAM
    (the slices of the experts it runs) and its multiply-accumulates; one multiply-accumulate is two operations
    of the TOPS figures, whatever the slice width;
  * a byte fetched from Flash is also written to DRAM once (1.5 pJ/bit on top of the 103); it is then read from
    DRAM like every other byte the computation uses;
  * energy adds up; latency: a missed slice has to arrive before its expert runs, so Flash time is serial, while
    DRAM reads stream under the computation: t = t_flash + max(t_dram, t_compute).
"""
from __future__ import annotations

PAPER = dict(dram_pj_per_bit=1.5, flash_pj_per_bit=103.0, dram_gbps=104.0, flash_gbps=10.0, tops=16.4,
             tops_per_watt=3.18)


def step_cost(flash_bytes: int, dram_bytes: int, macs: int, hw: dict = PAPER):
    """(energy in joules, latency in seconds) of one step."""
    flash_bits = 8.0 * flash_bytes
    dram_bits = 8.0 * dram_bytes
    ops = 2.0 * macs
    energy = flash_bits * hw["flash_pj_per_bit"] * 1e-12
    energy += (flash_bits + dram_bits) * hw["dram_pj_per_bit"] * 1e-12
    energy += ops / (hw["tops_per_watt"] * 1e12)
    t_flash = flash_bits / (hw["flash_gbps"] * 1e9)
    t_dram = dram_bits / (hw["dram_gbps"] * 1e9)
    t_compute = ops / (hw["tops"] * 1e12)
    return energy, t_flash + max(t_dram, t_compute)
