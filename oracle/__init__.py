"""CPU oracle of the KroQuant online quantizer -- TEST INFRASTRUCTURE ONLY.

``oracle.c_oracle`` wraps the plain C implementation (fp64 sums, OpenMP over
token rows); ``oracle.np_oracle`` is an independent NumPy restatement.  Neither
imports the CUDA package, and the CUDA package never imports this one: only the
tests, the smoke check and the bench's cpu_baseline / reference arm do.
"""
