"""CPU oracle of the HTTM global-attention path. Test infrastructure only."""
