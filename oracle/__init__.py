"""fp64 CPU oracle for the ClusterAttention hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this
package: it exists so that the tests, the smoke check and the benchmark's
CPU-baseline leg have a slow, plain, independently written statement of what
the paper's method computes.  It shares no code with the CUDA kernels.
"""
