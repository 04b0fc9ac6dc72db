"""CPU oracle of the CollectiveKV decode path.  TEST INFRASTRUCTURE ONLY.

Nothing under this package may be imported by the CUDA library or its Python
binding; only tests, the smoke check and the bench's CPU-baseline leg use it.
"""
