"""B200-native tiered decode hot path (BOOST, arxiv 2609.13592).

The product is the C-ABI library built from `csrc/` (see `include/boost.h`);
`binding` holds the thin ctypes layer over it and `synth` the seeded input
generators that tests, the smoke check and the benchmark share.  Importing the
package loads nothing heavy; `binding.lib()` loads the shared library and
raises if it has not been built.
"""
__all__ = ["binding", "synth"]
