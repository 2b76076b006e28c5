"""B200-native GWQ mixed-precision linear layer (arXiv 2411.00850).

`paper_2411_00850_b200.binding` wraps the C-ABI library (select, pack, linear);
`paper_2411_00850_b200.synth` draws the seeded synthetic inputs.
"""
