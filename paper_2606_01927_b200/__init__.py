"""B200-native batched token sampler (the sampling task T4 of arxiv 2606.01927).

``workloads`` holds the seeded synthetic input generators.  The sampler itself lives in
the CUDA library ``libalbireo_sample.so`` (sources under ``csrc/``) and is reached
through ``binding`` -- there is no CPU fallback: importing ``binding`` without the
built library raises.
"""
