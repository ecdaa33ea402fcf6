"""fp64 CPU oracle for paged decode attention and KV append.  Test infrastructure only."""
