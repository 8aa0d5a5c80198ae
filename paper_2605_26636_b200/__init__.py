"""JetViT token mixers for B200 (sm_100a): linear attention with squeeze dynamic
depth-wise convolution, 2D window attention, full softmax attention and the
per-layer L/W/F schedule driver, as hand-written CUDA behind a C ABI.

``paper_2605_26636_b200.jetvit`` is the ctypes binding (loaded on first use);
``paper_2605_26636_b200.inputs`` draws the seeded synthetic workloads.
"""
__version__ = "0.1.0"
