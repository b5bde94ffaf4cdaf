"""CPU oracle of the FreqDepthKV hot path.  Test infrastructure only: the product never imports it."""
