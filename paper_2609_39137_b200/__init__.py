"""B200-native MoE routing + load-control hot path of ID Balancing
(arXiv 2609.39137): thin Python binding over the CUDA C-ABI library.

`binding` marshals arguments only; every step of the path runs in the CUDA
kernels of libmoe_route_b200.so.  `synth` draws the seeded synthetic inputs.
Importing this package does not load the library; using `binding.Router`
without a built library raises.
"""
__all__ = ["binding", "synth", "build"]
