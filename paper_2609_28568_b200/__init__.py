"""B200-native dense linear layers (forward, dgrad, wgrad, dbias) behind a C ABI.

``binding`` marshals arguments to the CUDA library; ``synth`` makes seeded
inputs; ``shapes`` lists the layer shapes of the workloads. Nothing here
computes on the CPU: without the compiled CUDA library every call raises.
"""
__version__ = "0.1.0"
