"""CPU oracle for the Ouroboros verification path.

TEST INFRASTRUCTURE ONLY: a slow, plain fp64 restatement of what the CUDA library computes, written
from the paper.  Only tests, the smoke check and the benchmark's CPU-baseline leg may import it;
the product package never does, and the oracle never imports the product's kernels or binding.
"""
