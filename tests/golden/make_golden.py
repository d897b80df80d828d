"""Writes the stored checksums under tests/golden/.  Calls only the input generator and oracle/.

    python tests/golden/make_golden.py
"""
import os
import sys
import zlib

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import ring  # noqa: E402
from paper_2609_34334_b200 import workloads as W  # noqa: E402


def main():
    with open(os.path.join(HERE, "generator_crc.txt"), "w") as f:
        f.write("# crc32 of generator output bytes; written by tests/golden/make_golden.py\n")
        f.write("uniform_fp32_seed0_rank0_n4096 %08x\n" % zlib.crc32(W.uniform(0, 0, 4096, "fp32").tobytes()))
        f.write("normal_bf16_seed1_rank7_n4096 %08x\n" % zlib.crc32(W.normal(1, 7, 4096, "bf16", 1e-3).tobytes()))
        f.write("int_bf16_seed5_rank2_n4096 %08x\n" % zlib.crc32(W.small_integers(5, 2, 4096, "bf16").tobytes()))
    # oracle results on the two small benchmark configurations (guards against silent oracle changes)
    with open(os.path.join(HERE, "oracle_result_crc.txt"), "w") as f:
        f.write("# crc32 of rank 0's oracle result; written by tests/golden/make_golden.py (oracle/ only)\n")
        c1 = W.C1_SMALL_ALLREDUCE
        ys = ring.ring_allreduce(W.rank_inputs(c1.dist, c1.seed, c1.R, c1.count, c1.dtype))
        f.write("%s %08x\n" % (c1.name, zlib.crc32(ys[0].tobytes())))
        c2 = W.C2_DP_BUCKET
        ys = ring.ring_allreduce(W.rank_inputs(c2.dist, c2.seed, c2.R, c2.count, c2.dtype, c2.sigma))
        f.write("%s %08x\n" % (c2.name, zlib.crc32(ys[0].tobytes())))


if __name__ == "__main__":
    main()
