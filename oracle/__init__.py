"""float64 CPU oracle of the IDKM hot path.  Test infrastructure only: the product never imports it."""
