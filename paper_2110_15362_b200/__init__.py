"""B200-native sparse-bitmap activation codec (BitTrain's stash format).

`binding` exposes the C ABI of libbittrain.so (CUDA kernels for sm_100a);
`workloads` draws the seeded synthetic inputs; `build` compiles the library.
Nothing is loaded until `binding.lib()` is first called.
"""
__all__ = ["binding", "build", "workloads"]
