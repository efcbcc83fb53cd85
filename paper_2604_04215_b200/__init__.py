"""B200-native rollout denoising step for diffusion LLMs (C-ABI library + thin ctypes binding)."""
