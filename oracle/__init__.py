"""CPU oracle package -- TEST INFRASTRUCTURE ONLY.

Holds the plain definitions the GPU library is checked against:

* ``oracle.gemm``      -- the dense product with fp64 accumulation (C, OpenMP)
* ``oracle.taxonomy``  -- the paper's tiling taxonomy, data-volume formulas and
                          pipeline-latency formulas (pure Python)

Nothing here imports the GPU package and the GPU package never imports this.
"""
