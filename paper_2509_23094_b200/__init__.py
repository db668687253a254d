"""d2Cache decode step for B200: hand-written sm_100a CUDA behind a C ABI.

`paper_2509_23094_b200.binding` loads the shared library (and raises if it is
missing); `paper_2509_23094_b200.inputs` draws seeded synthetic inputs.  Nothing
heavy is imported here.
"""
