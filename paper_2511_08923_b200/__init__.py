"""TiDAR single-forward decode step for NVIDIA B200: CUDA library + thin ctypes binding."""
from .binding import Tidar, TidarError, attention_static, bf16_bits_to_f32, load, pack_weights, plan_ks  # noqa: F401
