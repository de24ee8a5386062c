"""B200 (sm_100a) library for the fused attention and fused Linear+bias+GELU operators.

``paper_2604_16498_b200.binding`` wraps the C ABI declared in ``include/forge.h``;
``paper_2604_16498_b200.workloads`` draws the seeded synthetic inputs.  Importing the
package does not load the CUDA library; the binding loads it on first use and raises
if it is missing (there is no fallback path).
"""
__all__ = ["binding", "workloads", "build"]
