"""B200-native flow-matching action-expert denoising loop (C-ABI library + thin binding).

Importing the package does not load the CUDA library; the binding loads it on first use and
raises if it is missing (there is no CPU fallback)."""
