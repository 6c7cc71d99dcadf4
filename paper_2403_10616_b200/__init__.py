"""B200-native module-wise outer synchronisation of DiPaCo (Algorithm 1, outer loop).

``paper_2403_10616_b200.binding`` wraps the C-ABI library ``libdipaco.so`` (CUDA, sm_100a);
``paper_2403_10616_b200.synth`` produces the seeded synthetic workloads.  The binding is loaded
on first use and raises if the CUDA library has not been built: there is no CPU path.
"""

__all__ = ["binding", "synth", "build"]
