"""B200-native n-wise interlocking-backpropagation training step (CUDA library + thin ctypes binding)."""
from .binding import (ILError, Model, lib, lr_schedule, nwise_streams, pipeline_transfers,  # noqa: F401
                      time_per_batch)
