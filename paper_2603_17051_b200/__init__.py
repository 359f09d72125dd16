"""Rolling-KV chunk attention for sm_100a: C-ABI library plus a thin ctypes binding.

``from paper_2603_17051_b200 import binding`` loads (and, when stale, builds) libastro.so.
Importing the package itself loads nothing.
"""
