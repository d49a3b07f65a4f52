"""B200-native budgeted MoE-layer forward (Alloc-MoE hot path).

`paper_2604_08133_b200.synth` draws the seeded synthetic inputs;
`paper_2604_08133_b200.binding` marshals arguments to the C-ABI library built
from `csrc/` (loaded on first use; there is no CPU fallback).
"""
