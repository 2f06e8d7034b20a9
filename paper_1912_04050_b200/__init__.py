"""B200-native Benes-network routing: switch-setting computation and payload apply.

The compute path is a C-ABI CUDA library (``include/benes.h``) built for
sm_100a; this package only marshals arguments to it.  There is no CPU
fallback: calling an operation without the built CUDA library raises.
"""
