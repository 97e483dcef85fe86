"""B200-native execution of GEMM-anchored fused DNN subgraphs (MLP chains and scaled-dot-product
attention blocks) behind a small C ABI: gc_partition_create / gc_compile / gc_execute.

Importing the package does not load the CUDA library; ``paper_2301_01333_b200.binding`` does, and
fails loudly if it has not been built."""
from .graph import Graph, LogicalTensor, Op  # noqa: F401
