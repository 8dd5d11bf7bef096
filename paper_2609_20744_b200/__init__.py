"""Bidirectional Video Delta Attention forward for NVIDIA B200 (sm_100a).

`paper_2609_20744_b200.binding` wraps the C-ABI shared library (hand-written CUDA);
`paper_2609_20744_b200.inputs` draws the seeded synthetic workloads.  Importing the
package itself loads neither torch nor the shared library.
"""

__all__ = ["binding", "inputs", "build"]
