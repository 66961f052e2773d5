"""B200-native batched CartPole step: C-ABI CUDA library + thin Python binding."""
