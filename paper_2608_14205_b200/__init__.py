"""B200-native FreeBalance hot path: residual workload prediction, budgeted
expert-swap planning and the dispatch index, as a C-ABI CUDA library with a thin
Python binding.  Importing the package does not load the CUDA library; the
binding does so on first use and raises if it is missing."""
