"""SANTA++ decode attention for NVIDIA B200 (sm_100a).

The CUDA library is loaded on first use by `paper_2609_35629_b200.binding`;
`paper_2609_35629_b200.synth` (seeded inputs) needs neither CUDA nor the library.
"""
__version__ = "0.1.0"
