"""B200-native graph VM for pruned computation graphs (arXiv 1707.08265).

``paper_1707_08265_b200.binding`` wraps the C-ABI library (``libdragon.so``);
``paper_1707_08265_b200.workloads`` writes the seeded synthetic graphs.
Nothing is loaded at import time.
"""
