"""B200-native checkpointed CNN training step (host planners + sm_100a kernels behind a C ABI)."""
