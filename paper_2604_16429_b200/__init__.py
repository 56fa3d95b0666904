"""MOSAIC mesh-aligned block-sparse attention, B200 (sm_100a) hot path.

The compute lives in ``csrc/`` behind a C ABI (``include/mosaic_bsa.h``);
``binding`` marshals arguments to it and nothing else.
"""
