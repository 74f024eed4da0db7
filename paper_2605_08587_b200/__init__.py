"""B200-native (sm_100a) Kaczmarz Linear Attention hot path: chunkwise forward and decode step."""
