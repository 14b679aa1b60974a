"""B200-native hot path of TapOut (arXiv 2511.02017): bandit-selected stop rules,
speculative-sampling verification and on-device arm updates over vocabulary-wide logits.

`paper_2511_02017_b200.binding` wraps the C-ABI library (libtapout.so, CUDA, sm_100a);
`paper_2511_02017_b200.synth_inputs` generates the seeded synthetic logits.
Importing the package loads nothing; the binding fails loudly if the library is missing.
"""
__all__ = ["binding", "synth_inputs"]
