"""B200-native (sm_100a) inference-time Mixture-of-Lookup-Experts layer (arXiv 2503.15798).

The product is the C-ABI library built from ``csrc/`` (declared in ``include/mole.h``);
``paper_2503_15798_b200.binding`` is its argument-marshalling Python face.  Importing the
package does not load the library; the first call through the binding does, and fails
loudly if the library has not been built.
"""

__all__ = ["binding", "inputs", "build"]
