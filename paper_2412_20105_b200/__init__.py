"""ST^3 decode-step attention over a trimmed visual KV cache, for NVIDIA B200 (sm_100a).

The product is the C library `libst3.so` (sources in `csrc/`, interface in `include/st3.h`);
`binding` is a thin ctypes layer over it with the same entry-point names.  Importing this
package loads nothing; `binding.load()` fails loudly if the library has not been built.
"""
