"""CPU oracle of the batched response-time analysis -- TEST INFRASTRUCTURE ONLY.

Nothing here is part of the product path.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; it shares no code with the CUDA library and never
imports it.

``rta``  ctypes wrapper of ``rta_oracle.c`` (the analysis, written from the paper's Sec. 6)
``sim``  ctypes wrapper of ``des_sim.c`` (a tick-level discrete-event simulator used to check
         that observed response times never exceed the analytic bounds)
"""
