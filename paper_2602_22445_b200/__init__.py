"""Batched B200 executor for the correction-based fault-tolerant reduce and allreduce."""
