"""CPU oracle for the dual-routed MWQ MoE layer.  TEST INFRASTRUCTURE ONLY.

Plain, slow numpy restatement of what the paper's method computes, written from the paper:
Matryoshka Weight Quantization (Section 3.3.1, Eq. 2 and Eq. 4, reconstruction rule below Eq. 5),
dual routing (Section 3.2 and the models of Section 5.1), the SwiGLU expert FFN and the weighted
combine.  Values are fp64; arithmetic that decides an integer (codes, indices, widths) is fp32 in
a pinned order so that it can be compared bit for bit.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` / ``--impl reference`` legs
of ``bench.py`` may import this package.  It shares no code with the CUDA path and never imports
it; the product path never imports this.

Parity unpinned (the paper gives no worked example or size to check against, the reading is
stated in the function's docstring): ``routing.bit_width_choice`` (architecture of the bit-width
router, argmax selection, no scaling of the expert output by the router probability).
"""
