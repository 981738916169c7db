"""B200-native GP-EI candidate scoring for the Bayesian-optimisation layer of R^3.

The product is the C-ABI library ``libr3gp.so`` (hand-written sm_100a CUDA);
``binding`` marshals arguments to it and ``workloads`` draws the seeded
synthetic inputs.  Importing the package does not load the library; the first
call into ``binding`` does, and fails loudly if it is missing.
"""
__version__ = "0.1.0"
