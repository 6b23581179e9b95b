"""B200-native KVCrush compression pass: score -> signature -> select -> compact.

The CUDA library is loaded on first use (``binding.lib()``); importing the
package, or its ``inputs`` module, does not need a GPU.
"""
