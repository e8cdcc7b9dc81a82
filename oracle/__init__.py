"""CPU reference oracle for the Local AdaAlter hot path (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  The CUDA library never does.
"""
