"""B200-native BFP8 paged decode attention (deferred dequantization, paper section 3.3).

`paper_2606_29986_b200.hma` is the ctypes binding of the C-ABI library;
`paper_2606_29986_b200.synth` makes seeded synthetic inputs.  Nothing is loaded at import.
"""
