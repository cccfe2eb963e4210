"""fp64 CPU oracle for span-restricted decode attention.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this
package: it exists so that the tests, the smoke check and the benchmark's
CPU-baseline leg have an independent statement of what the method computes.
It shares no code with the CUDA library.
"""
