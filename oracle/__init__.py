"""Oracle for the C-Coll hot path: TEST INFRASTRUCTURE ONLY (tests, smoke check, CPU-baseline timing).

The product package never imports this; see ccz_oracle.h for what it follows in the paper.
"""
