"""B200-native mixed-adapter LoRA apply (dense projections and packed MoE
expert LoRA) behind a C-ABI CUDA library; see include/mint_lora.h.

`binding` loads libmint_lora.so (no CPU fallback), `synth` draws the seeded
workloads, `harness` uploads them, `build` compiles the library."""
