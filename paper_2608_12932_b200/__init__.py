"""B200-native W4A8 quantized linear (Sec. 3.4 of the FlashDrive paper)."""
