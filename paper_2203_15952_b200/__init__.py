"""B200-native quantized linear layer (native integer quantization, arXiv 2203.15952).

`binding` holds the Python names of the C ABI (include/aqt.h); `encoder` chains layers into the
Conformer-shaped workloads; `inputs` generates the seeded synthetic tensors.  Importing this
package loads nothing; the CUDA library is loaded on the first call into `binding`.
"""
__all__ = ["binding", "build", "encoder", "inputs"]
