"""B200-native Token-Level Intersection (TLI) verification.

``paper_2502_05202_b200.tli`` binds the CUDA library (C ABI in include/tli.h);
``paper_2502_05202_b200.workload`` draws the seeded synthetic inputs;
``paper_2502_05202_b200.build`` compiles the library.  Importing the package
itself loads nothing.
"""
