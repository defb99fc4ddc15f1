"""TEST INFRASTRUCTURE: CPU reference of the n-softsync parameter-server update.

Imported only by the tests, the smoke check and the benchmark's CPU-baseline
leg.  Never by the product package.
"""
