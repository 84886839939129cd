"""Plain CPU restatement of the VIA-SD verification cycle, written from the paper.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product never routes through it and the two
share no code.
"""
