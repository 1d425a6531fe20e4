"""fp64 CPU oracle for the LAQ re-eviction step (Section 4.3, Eq. 4). Test infrastructure only:
nothing on the product path may import this package."""
