"""CPU oracle for the KV-block rotation path.  TEST INFRASTRUCTURE, not product code.

Only ``tests/``, the smoke check and the bench's CPU-baseline / reference arm may
import this package.  It shares no code with the CUDA library and never imports it.

Modules
-------
kv_definition  the definition written out three ways: 6-D numpy indexing, flat
               element-by-element index arithmetic (tiny cases), and a symbolic
               content-tag model.
kv_oracle      ctypes front end of ``kv_oracle.c`` (byte arrays + memcpy of one
               segment at a time; also the multi-threaded variant that is timed).
build          compiles ``kv_oracle.c`` with gcc.
"""
