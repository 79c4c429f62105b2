"""B200-native visual-token reduction of CoVSpec (Sec. III-A): a C-ABI CUDA library plus this
thin binding.  `workloads` (seeded synthetic inputs) imports without the compiled library; the
binding in `api` fails loudly when the library is missing."""
