"""CPU oracle for the D3ToM merge-layer path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this
package; only the test-suite, the smoke check and the benchmark's CPU
baseline leg call it.  It shares no code with the CUDA path.
"""
