"""CPU checker for the paged-KVCache transfer path (test infrastructure only)."""
