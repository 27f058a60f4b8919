"""B200-native Softmax Linear Attention hot path (chunkwise gated linear attention with
head-level softmax gates): a C-ABI CUDA library plus a thin Python binding."""
