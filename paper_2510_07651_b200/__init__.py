"""B200-native OBCache score / select / compact library (Python binding over the C-ABI)."""
