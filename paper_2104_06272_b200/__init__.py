"""Anakin hot path (co-located env step + act + learn) as hand-written sm_100a CUDA kernels behind a
C-ABI library.  Importing the package loads nothing; `paper_2104_06272_b200.binding` loads the library
and fails loudly if it has not been built."""
