"""B200-native vocabulary-side hot path of the entropy-holding RL method
(temperature softmax statistics, Gumbel-max sampling, masked mean entropy,
group advantages) behind a C-ABI CUDA library.

``paper_2505_18573_b200.binding`` is the thin ctypes layer over ``libe3.so``;
``paper_2505_18573_b200.inputs`` holds the seeded synthetic input generators.
Nothing here falls back to a CPU implementation: without the built CUDA
library every call raises.
"""
