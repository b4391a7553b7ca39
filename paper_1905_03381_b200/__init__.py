"""B200-native AutoAssist instance-shrinking batch generator (arXiv 1905.03381).

The product is the C-ABI CUDA library declared in ``include/autoassist.h``;
``binding`` marshals torch tensors into it and ``workloads`` draws the seeded
synthetic inputs.  Importing the package does not load the CUDA library; the
first call into ``binding`` does, and fails loudly if it has not been built.
"""
