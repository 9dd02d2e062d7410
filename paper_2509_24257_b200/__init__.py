"""B200-native verifier prefill for VeriLLM: Python binding over the C-ABI library."""
