"""B200-native hot path of PODS (Policy Optimization with Down-Sampling, arxiv 2504.13818).

``paper_2504_13818_b200.binding`` wraps the C-ABI CUDA library (``include/pods.h``);
``paper_2504_13818_b200.workloads`` draws the seeded synthetic inputs.  Importing the
package loads nothing; the CUDA library is loaded on first use and its absence is an error.
"""
__version__ = "0.1.0"
