"""TEST INFRASTRUCTURE: CPU checker for the flow-control simulator (see fcsim_oracle.cpp).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
