"""B200-native fused draft+verify step for diffusion-AR self-speculation.

The CUDA library is loaded lazily by ``paper_2609_34388_b200.binding``; importing the
package itself (for instance to reach the synthetic input generators) loads no
native code.
"""
__all__ = ["binding", "synth"]
