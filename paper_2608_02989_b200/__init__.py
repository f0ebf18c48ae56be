"""B200-native AcceptMoE verifier-side MoE layer (one verification block per call).

``paper_2608_02989_b200.acm`` is the Python binding of the C-ABI library in ``csrc/``;
``paper_2608_02989_b200.workloads`` generates the seeded synthetic inputs.
"""
