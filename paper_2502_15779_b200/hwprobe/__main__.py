"""Micro-benchmarks behind the kernel design: what the B200's pipes do with the operations the W2A4 GEMV is made of.

    python -m paper_2502_15779_b200.hwprobe [pipes] [umma_rate] [umma_pipeline] [sign_field_mix] [bmma_rate]

builds the named programs (all by default) with nvcc for sm_100a next to their sources and runs them on the
current GPU; each prints its own table. They measure, they do not test anything: every wait in them is bounded.

  pipes           issue rates of LOP3, dp4a and int8 mma.sync alone and combined (other warps, same warp, with and
                  without a dependency): does the legacy tensor path overlap with the logic pipe?
  umma_rate       clocks per tcgen05.mma kind::i8 (M = 128, K = 32) for N = 8 .. 256, A from tensor or shared memory
  umma_pipeline   the whole tcgen05 route for this GEMV: masked code words written to tensor memory by the threads,
                  int8 activations in shared memory, sums checked against the host, bytes of weights per clock
  sign_field_mix  the instruction mix of a formulation with fewer logic operations but more shifts and adds
  bmma_rate       clocks per binary mma.sync (m16n8k256, and.popc) and a check of its fragment layout
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
PROGRAMS = {"pipes": [[]], "umma_rate": [[]], "sign_field_mix": [[]], "bmma_rate": [[]],
            "umma_pipeline": [["1", "4", "1", "0"], ["8", "8", "1", "0"], ["1", "2000", "148", "0"], ["8", "2000", "148", "0"],
                              ["1", "2000", "148", "1"], ["1", "2000", "148", "2"]]}


def main():
    names = sys.argv[1:] or list(PROGRAMS)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    for n in names:
        exe = os.path.join(HERE, n)
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-o", exe,
                               os.path.join(HERE, n + ".cu")])
        for args in PROGRAMS[n]:
            subprocess.check_call([exe] + args)


if __name__ == "__main__":
    main()
