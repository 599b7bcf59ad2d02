"""fp64 CPU oracle of the SVD-Cache hot path.  Test infrastructure only: the product
package never imports it (see ``svdcache_oracle.c`` for what it computes and its pins)."""
