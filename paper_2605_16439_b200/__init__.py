"""KVCapsule decode-time hot path for B200 (sm_100a): C-ABI CUDA library + thin binding."""
