"""TEST INFRASTRUCTURE -- the CPU oracle of the integer convolution layer.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline leg of ``bench.py`` may
import this package.  It shares no code with the CUDA path and never imports it.
"""
