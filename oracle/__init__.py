"""CPU oracle for the VidKV hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this
package: it is a slow, plain restatement of the paper's algorithms that the
tests, the smoke check and the benchmark's CPU-baseline leg compare against.
It shares no code with the CUDA path.
"""
