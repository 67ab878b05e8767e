"""SOAR NVFP4 weight quantizer for NVIDIA B200: Python binding of the C-ABI library."""
