"""AdaScale SGD gain-ratio step for NVIDIA B200 (sm_100a).

``binding`` wraps the C-ABI CUDA library; ``synthetic`` draws seeded inputs.
"""
