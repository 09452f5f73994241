"""B200-native speculative-step hot path of Re-SpS (draft-tree construction, tree-masked
verification attention, greedy verify/accept, KV-cache compaction) behind a C-ABI library.

`binding` wraps the library (CUDA only; no fallback), `synth` generates the seeded synthetic
workloads, `build` compiles the library in-tree."""
