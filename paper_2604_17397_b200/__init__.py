"""B200-native hot path of SDVG block-autoregressive video diffusion (C-ABI library + thin binding)."""
