"""B200-native SeerAttention prefill hot path: AttnGate scores -> block index
lists -> causal GQA block-sparse attention, as hand-written sm_100a CUDA behind
a C ABI (`include/seer.h`).  `binding` is the ctypes layer over that ABI,
`workloads` draws the seeded synthetic inputs, `sharding` splits a layer by
KV head across ranks."""
