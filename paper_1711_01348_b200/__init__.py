"""B200-native evaluation of element-wise defined tensor expressions and of their derivative
expressions (Urban & van der Smagt, 2017).  Everything runs in libtad.so; this package is the
ctypes binding."""
from .binding import (AccessInfo, KernelStats, Plan, TadError, extended_euclid,  # noqa: F401
                      fourier_motzkin, measure_fp32_rate, smith_normal_form, lib, EXPORTS)
