"""TEST INFRASTRUCTURE -- the CPU oracle for paged-KV pack/unpack.

Only tests, the smoke check and the CPU-baseline leg of the benchmark import
this package.  It shares no code with the CUDA library and never imports it.
"""
