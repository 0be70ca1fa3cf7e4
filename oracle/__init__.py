"""CPU oracle for the distribution-aware fused-MoE path.

TEST INFRASTRUCTURE ONLY: a plain, slow, fp64 restatement of what the paper
defines.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import it; it shares no code with the CUDA library.
"""
