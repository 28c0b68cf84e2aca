"""B200-native GLIDE hybrid attention (sliding-window softmax + linear recurrent state, one shared normaliser).

The compute lives in the CUDA library behind the C ABI declared in include/glide.h;
`paper_2607_24788_b200.glide` is the thin ctypes binding. There is no CPU fallback:
loading the binding without the built library raises.
"""
