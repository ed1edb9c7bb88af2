"""B200-native (sm_100a) hot path of one TwIST training round.

The CUDA library is loaded lazily on first use (see `binding`); importing the
package itself touches neither CUDA nor the shared library, so the input
generators in `inputs` can be used on machines without a GPU.
"""
