"""B200-native AIF pre-ranking scoring pass: a C-ABI CUDA library plus a thin Python binding.

`synth` (input generator) imports no native code; `binding` loads the CUDA library and fails loudly when it
is missing."""

__all__ = ["synth", "binding"]
