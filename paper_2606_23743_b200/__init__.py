"""B200-native block-sparse spatiotemporal attention (sm_100a CUDA behind a C ABI).

The CUDA library is loaded on first use of :mod:`paper_2606_23743_b200.binding`; importing
the package itself needs neither a GPU nor the built extension.
"""
