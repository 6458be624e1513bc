"""B200-native OSC dual-path quantized linear layer (C-ABI library + thin binding).

`paper_2604_12782_b200.binding` loads the CUDA library and fails loudly if it
is missing; `synth` and `roofline` are host-only helpers and import nothing else.
"""
