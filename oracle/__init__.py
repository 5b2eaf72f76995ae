"""TEST INFRASTRUCTURE — CPU oracle of the edge-feature join (see ccr_oracle.cpp for what it follows).

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs import this package.
"""
