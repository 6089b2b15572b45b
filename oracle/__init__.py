"""CPU oracle (test infrastructure): literal simulation of the paper's reduce / allreduce."""
