"""PackCache hot path for one B200: budget plan, token scoring + per-frame top-k, gather/pack and per-frame
attention over the compacted KV cache, as CUDA kernels behind a C ABI (see ``include/packcache.h``)."""
