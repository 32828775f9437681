"""CPU oracle of the FlashCache compression path (test infrastructure only)."""
