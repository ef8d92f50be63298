"""B200-native verify/correct, acceptance head and stop rule of SpecDec++ (arXiv 2405.19715).

`paper_2405_19715_b200.specdec` is the binding of the C-ABI library (include/specdec.h);
`paper_2405_19715_b200.workloads` draws the seeded synthetic inputs.  Importing the package
loads nothing; the CUDA library is loaded (and built if stale) on first use of the binding.
"""
