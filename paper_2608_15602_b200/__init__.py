"""B200-native FluxBin decode linear layer (y = What x, LUT GEMV) behind a small C-ABI.

`paper_2608_15602_b200.synth` holds the seeded input generators (numpy only).
`paper_2608_15602_b200.fluxbin` is the thin ctypes binding of csrc/ (loaded on first use).
"""
