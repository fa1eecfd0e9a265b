"""B200-native Finch KV-cache compression step: score -> select -> compact behind a C ABI (libfinch.so).

``binding`` holds the ctypes entry points (same names as include/finch.h), ``workloads`` the seeded synthetic
inputs, ``build`` the nvcc build of the library.  Nothing here computes on the CPU.
"""
