"""B200-native hot path of the Sparsely-Gated Mixture-of-Experts layer.

`binding` wraps the C-ABI CUDA library (argument marshalling only); `synth` draws the
seeded synthetic workloads. Importing the package loads no native code; the first use of
`binding` does, and fails loudly if the library has not been built.
"""
