"""B200-native decode of XOR-gate-network encrypted weight bit-planes, fused with the
sparse quantized product that consumes them.

``paper_1905_10138_b200.sqnn`` is the thin binding over the C-ABI CUDA library;
``paper_1905_10138_b200.workloads`` draws the seeded synthetic layers.  Importing the
package does not load the CUDA library; using ``sqnn`` without it raises.
"""
