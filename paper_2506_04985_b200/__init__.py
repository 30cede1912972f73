"""B200-native statically quantised W4A4 linear path (FPTQuant, Sec. 3 / App. B, J).

`paper_2506_04985_b200.binding` loads the C-ABI shared library and exposes its
entry points under the same names; `paper_2506_04985_b200.synth` draws the seeded
synthetic inputs.  Importing the package itself loads nothing.
"""
__all__ = ["binding", "synth"]
