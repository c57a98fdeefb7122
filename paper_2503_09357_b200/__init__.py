"""Batched evaluation of candidate parallel plans on B200 (C-ABI library + ctypes binding).

`binding` holds the entry points of include/pe.h under the same names; `workloads`
holds the seeded synthetic inputs.  Importing `binding` requires the built libpe.so.
"""
