"""B200-native speculate-and-verify step (suffix index, draft trees, tree-masked verify attention, accept).

Importing the package does not load the CUDA library; `paper_2607_17299_b200.binding` does, and fails
loudly when the library has not been built."""
