"""Decode-phase attention over a long fp16 KV cache, hand-written for sm_100a.

`binding` is the thin ctypes layer over the C-ABI library (it raises if the library has not
been built); `workloads` draws the seeded synthetic inputs; `build` compiles the library.
"""
