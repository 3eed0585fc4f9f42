"""CDL quantized layer on B200 (package under construction: inputs only so far)."""
