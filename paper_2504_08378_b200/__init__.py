"""B200-native active-weight selection and sparse GEMV (ActiveFlow decoding hot path).

``paper_2504_08378_b200.afx`` is the binding over the C-ABI CUDA library;
``paper_2504_08378_b200.synth`` draws the seeded synthetic inputs.
"""
