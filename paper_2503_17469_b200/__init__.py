"""B200-native weighted gradient aggregation, fused update and batch-size controller (OmniLearn).

``paper_2503_17469_b200.binding`` is the Python face of the C-ABI library (loaded on first use);
``paper_2503_17469_b200.workloads`` holds the seeded synthetic inputs.
"""
