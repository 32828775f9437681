"""B200-native FlashCache compression path (score -> allocate -> select -> compact).

The CUDA library is loaded on first use of `paper_2511_16786_b200.binding`;
importing the package alone (for example to reach the input generator in
`synth_kv`) needs no GPU and no built extension.
"""
__all__ = ["binding", "synth_kv", "build"]
