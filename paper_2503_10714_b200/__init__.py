"""B200 (sm_100a) compressed-KV decode path of ZSMerge behind a C ABI (libzsm.so).

`build` compiles the library; `binding` exposes its entry points one to one.
"""
