"""B200-native quantised verification pass (Quasar, arXiv 2603.01399).

`paper_2603_01399_b200.binding` wraps the C-ABI library `libquasar.so`
(argument marshalling only); `paper_2603_01399_b200.synth` draws the seeded
synthetic inputs.  Importing this package does not load the CUDA library;
`binding.lib()` does and raises if it has not been built.
"""
